"""The fixed-scratch BinGrad-b entry point against the regular one.

Some users of this library run where device allocation is not theirs to do: a gradient hook that
fires in the middle of a step, or a process whose memory pool another framework owns.  They call
ogq_levels_bingrad_b_noalloc, which keeps the solver's counters in an array built into the library.
This file checks that it gives the same levels, thresholds and status words as ogq_levels_bingrad
(same tolerance as the other level tests: 1e-5 of the tensor's largest level), on two calls in a row
that reuse the built-in array with different buckets, at the largest tensor count it accepts, that it
leaves the amount of device memory in use unchanged, and that it refuses more tensors than it holds.
It is collected last on purpose, and it also passes when run alone in a fresh process.
"""
import numpy as np
import pytest
import torch

import ogq_workloads as wl
import paper_2002_11082_b200 as ogq

pytestmark = pytest.mark.gpu


def _bucket(seed):
    r = np.random.Generator(np.random.PCG64(seed))
    sizes = [70001, 0, 1, 5, 4097, 262147, 33, 1 << 20]
    parts = [wl.laplace(r, n, 10.0 ** r.uniform(-5, -2)) if n else np.zeros(0, np.float32) for n in sizes]
    return np.concatenate(parts), wl.offsets_from_sizes(sizes)


def _run_both(vals, h_off, lloyd):
    dev = torch.device("cuda:0")
    T, N = h_off.size - 1, int(h_off[-1])
    grad = torch.from_numpy(vals).to(dev)
    off = torch.from_numpy(h_off).to(dev)
    out = {}
    for name in ("regular", "noalloc"):
        lv = torch.full((T, 2), float("nan"), device=dev)
        th = torch.full((T,), float("nan"), device=dev)
        st = torch.full((T,), -1, dtype=torch.int32, device=dev)
        if name == "regular":
            ws_bytes = ogq.ogq_workspace_bytes(T, N, 3)
            ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
            ogq.ogq_levels_bingrad(grad, off, T, N, ogq.OGQ_BINGRAD_B, lloyd, lv, th, st, ws, ws_bytes)
        else:
            ogq.ogq_levels_bingrad_b_noalloc(grad, off, T, N, lloyd, lv, th, st)
        torch.cuda.synchronize()
        out[name] = (lv.cpu().numpy(), th.cpu().numpy(), st.cpu().numpy())
    return out


def _assert_same(out):
    (lv_a, th_a, st_a), (lv_b, th_b, st_b) = out["regular"], out["noalloc"]
    assert np.array_equal(st_a, st_b)
    for t in range(lv_a.shape[0]):
        tol = 1e-5 * float(np.max(np.abs(lv_a[t])))
        assert np.all(np.abs(lv_a[t].astype(np.float64) - lv_b[t]) <= tol), t
        assert abs(float(th_a[t]) - float(th_b[t])) <= tol, t


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    # first call: a big ragged bucket, mean-split levels
    vals, h_off = _bucket(21)
    _assert_same(_run_both(vals, h_off, 0))
    # second call reuses the built-in array: fewer tensors, other data, Lloyd updates
    b = wl.config2()
    _assert_same(_run_both(b.values, b.offsets, 3))


def test_noalloc_at_its_capacity_then_a_small_call():
    """T = 1024 puts the per-tensor counters at the far end of the built-in array; the small call that
    follows must not be disturbed by what the large one left there."""
    r = np.random.Generator(np.random.PCG64(31))
    sizes = [int(x) for x in r.integers(0, 3000, 1024)]
    sizes[5] = sizes[700] = sizes[1023] = 0
    sizes[17] = 300001
    parts = [wl.laplace(r, n, 10.0 ** r.uniform(-5, -2)) if n else np.zeros(0, np.float32) for n in sizes]
    _assert_same(_run_both(np.concatenate(parts), wl.offsets_from_sizes(sizes), 2))
    vals, h_off = _bucket(22)
    _assert_same(_run_both(vals, h_off, 1))


def test_noalloc_call_leaves_device_memory_in_use_unchanged():
    """What the entry point is for: the free device memory the driver reports is the same before and
    after calls (outputs and inputs are allocated by the test beforehand; torch's caching allocator
    is not asked for anything in between)."""
    dev = torch.device("cuda:0")
    vals, h_off = _bucket(23)
    T, N = h_off.size - 1, int(h_off[-1])
    grad = torch.from_numpy(vals).to(dev)
    off = torch.from_numpy(h_off).to(dev)
    lv = torch.zeros((T, 2), device=dev)
    th = torch.zeros(T, device=dev)
    st = torch.zeros(T, dtype=torch.int32, device=dev)
    ogq.ogq_levels_bingrad_b_noalloc(grad, off, T, N, 0, lv, th, st)  # first call: address lookup
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info(dev)
    reserved0 = torch.cuda.memory_reserved(dev)
    for _ in range(3):
        ogq.ogq_levels_bingrad_b_noalloc(grad, off, T, N, 2, lv, th, st)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info(dev)
    assert free1 == free0 and torch.cuda.memory_reserved(dev) == reserved0


def test_noalloc_rejects_more_tensors_than_it_holds():
    dev = torch.device("cuda:0")
    T = 1025
    h_off = np.arange(T + 1, dtype=np.int64) * 8
    grad = torch.zeros(int(h_off[-1]), device=dev)
    off = torch.from_numpy(h_off).to(dev)
    lv = torch.zeros((T, 2), device=dev)
    th = torch.zeros(T, device=dev)
    st = torch.zeros(T, dtype=torch.int32, device=dev)
    with pytest.raises(ogq.OgqError) as e:
        ogq.ogq_levels_bingrad_b_noalloc(grad, off, T, int(h_off[-1]), 0, lv, th, st)
    assert e.value.code == 5
    torch.cuda.synchronize()
