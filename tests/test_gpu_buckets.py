"""Fixed-length bucket mode (ogq_bucket_encode) against the oracle and against the per-tensor calls.

The oracle side is the per-tensor oracle applied to offsets j * d: the paper's bucket-based
quantization is the same method on equal slices of the flattened gradient (Section "Experiments").
"""
import numpy as np
import pytest
import torch

import oracle
import ogq_workloads as wl
import paper_2002_11082_b200 as ogq

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_helpers import DeviceBucket

SCHEME_OF = {"orq": (ogq.OGQ_ORQ, oracle.ORQ), "b": (ogq.OGQ_BINGRAD_B, oracle.B), "pb": (ogq.OGQ_BINGRAD_PB, oracle.PB)}


def bucket_offsets(total, d):
    nb = (total + d - 1) // d
    off = np.minimum(np.arange(nb + 1, dtype=np.int64) * d, total)
    return off


def run_encode(values, d, scheme, s, iters=0, seed=1, stream_id=0, clip_c=0.0):
    dev = torch.device("cuda:0")
    total = int(values.size)
    nb = (total + d - 1) // d
    bits = ogq.ogq_bits_for_levels(s)
    words = ogq.ogq_bucket_packed_words(total, d, bits)
    grad = torch.from_numpy(np.ascontiguousarray(values, np.float32)).to(dev)
    lv = torch.full((nb, s), float("nan"), device=dev)
    th = torch.full((nb,), float("nan"), device=dev)
    st = torch.full((nb,), -1, dtype=torch.int32, device=dev)
    pad = 64
    buf = torch.full((words + 2 * pad,), 0x5A5A5A5A, dtype=torch.int32, device=dev)
    ogq.ogq_bucket_encode(grad, total, d, scheme, s, iters, clip_c, seed, stream_id, lv, th, st, buf[pad : pad + words])
    torch.cuda.synchronize()
    h = buf.cpu().numpy().view(np.uint32)
    assert np.all(h[:pad] == 0x5A5A5A5A) and np.all(h[pad + words :] == 0x5A5A5A5A), "canary overwritten"
    return lv.cpu().numpy(), th.cpu().numpy(), st.cpu().numpy(), h[pad : pad + words].copy()


def close(got, want):
    tol = 1e-5 * float(np.max(np.abs(want))) if want.size else 0.0
    return bool(np.all(np.abs(got.astype(np.float64) - want.astype(np.float64)) <= tol))


def check_against_oracle(values, d, kind, s, iters=0):
    g_scheme, o_scheme = SCHEME_OF[kind]
    off = bucket_offsets(values.size, d)
    lv, th, st, packed = run_encode(values, d, g_scheme, s, iters, seed=9, stream_id=3)
    assert ogq.ogq_bucket_packed_words(values.size, d, ogq.ogq_bits_for_levels(s)) == int(
        oracle.packed_layout(off, oracle.bits_for(s))[-1])
    nb = off.size - 1
    if kind == "orq":
        w_lv, w_st = oracle.bucket_levels_orq(values, off, s)
        if iters:
            for j in range(nb):
                w_lv[j], _ = oracle.refine_orq(values[off[j] : off[j + 1]], w_lv[j], iters)
        # levels are data values: equal bit for bit except where T falls on an integer within rounding
        same = np.all(lv == w_lv, axis=1)
        assert same.mean() > 0.999, same.mean()
        for j in np.nonzero(~same)[0]:
            assert close(lv[j], w_lv[j]) or abs(
                oracle.expected_error(values[off[j] : off[j + 1]], lv[j])
                - oracle.expected_error(values[off[j] : off[j + 1]], w_lv[j])
            ) <= 1e-9 * oracle.expected_error(values[off[j] : off[j + 1]], w_lv[j]), j
        assert np.array_equal(st, w_st)
        th_in = None
    else:
        w_lv, w_th, w_st = oracle.bucket_levels_bingrad(values, off, o_scheme, iters)
        assert np.array_equal(st, w_st)
        ok = (w_st & ogq.OGQ_ST_NONFINITE) == 0  # BinGrad-b levels of a non-finite bucket are unspecified
        for j in np.nonzero(ok)[0]:
            assert close(lv[j], w_lv[j]), (j, lv[j], w_lv[j])
        if kind == "b":
            assert np.all(np.abs(th.astype(np.float64) - w_th)[ok] <= 1e-5 * np.abs(w_lv).max(axis=1)[ok] + 1e-30)
        th_in = th if kind == "b" else None
    # codes: bit-exact with both sides on the levels the GPU returned
    want, _ = oracle.bucket_quantize_pack(values, off, o_scheme, s, lv, th_in, 9, 3)
    assert np.array_equal(packed, want)
    return lv


@pytest.mark.parametrize("d", [128, 512, 2048, 32768])
def test_bucket_mode_on_resnet50_values(d):
    b = wl.resnet50_bucket(0)
    n = b.total if d >= 512 else 4_000_000  # 200 k oracle calls at d = 128 would only add minutes
    v = b.values[:n]
    check_against_oracle(v, d, "orq", 9)
    check_against_oracle(v[: 2_000_000 + 77], d, "orq", 3)
    check_against_oracle(v[: 2_000_000 + 77], d, "b", 2)
    check_against_oracle(v[: 1_000_000 + 130], d, "pb", 2)


@pytest.mark.parametrize("s", [5, 17])
def test_bucket_mode_other_level_counts_and_ragged_ends(s):
    v = wl.student_t(np.random.Generator(np.random.PCG64(40 + s)), 300_000 + 1, 3.0, 1e-3)
    for d in (256, 4096, 8192):
        check_against_oracle(v, d, "orq", s)
    check_against_oracle(v[:131], 128, "orq", s)  # one full bucket and a 3-element one
    check_against_oracle(v[:5], 128, "orq", s)


def test_bucket_mode_equals_the_per_tensor_calls_with_offsets_jd():
    v = wl.resnet50_bucket(0).values[5_000_000:5_600_000]
    for d in (512, 8192):
        off = bucket_offsets(v.size, d)
        db = DeviceBucket(v, off)
        for s in (3, 9):
            lv, _, st, packed = run_encode(v, d, ogq.OGQ_ORQ, s, 0, seed=4, stream_id=1)
            g_lv, g_st = db.levels_orq(s)
            assert np.array_equal(lv, g_lv) and np.array_equal(st, g_st)
            g_pk, _ = db.quantize_pack(ogq.OGQ_ORQ, s, g_lv, None, 4, 1)
            assert np.array_equal(packed, g_pk)


def test_bucket_mode_refinement_sweeps_follow_the_oracle_and_reduce_the_error():
    v = wl.resnet50_bucket(0).values[9_000_000:9_400_000]
    d = 2048
    off = bucket_offsets(v.size, d)
    greedy = check_against_oracle(v, d, "orq", 9, iters=0)
    for iters in (1, 50):
        refined = check_against_oracle(v, d, "orq", 9, iters=iters)
        e0 = sum(oracle.expected_error(v[off[j] : off[j + 1]], greedy[j]) for j in range(off.size - 1))
        e1 = sum(oracle.expected_error(v[off[j] : off[j + 1]], refined[j]) for j in range(off.size - 1))
        assert e1 < e0
    check_against_oracle(v[:100_000], 16384, "orq", 5, iters=20)  # the path without prefix sums


def test_bucket_mode_special_buckets_and_argument_checks():
    r = np.random.Generator(np.random.PCG64(50))
    v = wl.laplace(r, 6 * 256, 1e-3)
    v[256:512] = np.float32(0.25)          # constant bucket
    v[512 + 7] = np.float32(np.inf)        # non-finite bucket
    v[768:1024] = 0.0                      # all zeros
    v[1024:1280] = np.where(r.random(256) < 0.5, np.float32(-1.0), np.float32(2.0))  # two values only
    for kind, s in (("orq", 9), ("orq", 3), ("b", 2), ("pb", 2)):
        check_against_oracle(v, 256, kind, s)
    dev = torch.device("cuda:0")
    z = torch.zeros(1024, device=dev)
    i = torch.zeros(64, dtype=torch.int32, device=dev)
    for bad_d in (64, 100, 65536, 130):
        with pytest.raises(ogq.OgqError) as e:
            ogq.ogq_bucket_encode(z, 1024, bad_d, ogq.OGQ_ORQ, 9, 0, 0.0, 0, 0, z, z, i, i)
        assert e.value.code == 2
    with pytest.raises(ogq.OgqError):
        ogq.ogq_bucket_encode(z, 1024, 128, ogq.OGQ_ORQ, 4, 0, 0.0, 0, 0, z, z, i, i)
    ogq.ogq_bucket_encode(z, 0, 128, ogq.OGQ_ORQ, 9, 0, 0.0, 0, 0, z, z, i, i)  # nothing to do
    torch.cuda.synchronize()


@pytest.mark.parametrize("s,d", [(9, 512), (3, 2048), (5, 256), (17, 128), (2, 1024)])
def test_bucket_decode_sum_equals_unpack_sum_with_offsets_jd(s, d):
    """K workers encoded in bucket mode, summed by ogq_bucket_decode_sum: equal to the oracle's sum over
    the same packed buffers and to ogq_unpack_sum called with offsets j * d (bit for bit: same additions)."""
    dev = torch.device("cuda:0")
    K = 5
    total = 300_000 + 77
    off = bucket_offsets(total, d)
    scheme = ogq.OGQ_BINGRAD_B if s == 2 else ogq.OGQ_ORQ
    lvs, pks = [], []
    for k in range(K):
        v = wl.laplace(np.random.Generator(np.random.PCG64(90 + k)), total, 1e-3 * (1 + k))
        lv, th, st, packed = run_encode(v, d, scheme, s, 0, seed=2, stream_id=k)
        lvs.append(lv)
        pks.append(packed)
    d_lv = [torch.from_numpy(l).to(dev) for l in lvs]
    d_pk = [torch.from_numpy(p.view(np.int32)).to(dev) for p in pks]
    pad = 64
    buf = torch.full((total + 2 * pad,), 12345.0, device=dev)
    ogq.ogq_bucket_decode_sum(ogq.device_pointer_array(d_pk), ogq.device_pointer_array(d_lv), K, total, d, s, 1.0 / K,
                              buf[pad : pad + total])
    torch.cuda.synchronize()
    h = buf.cpu().numpy()
    assert np.all(h[:pad] == 12345.0) and np.all(h[pad + total :] == 12345.0), "canary overwritten"
    got = h[pad : pad + total]
    want = oracle.bucket_unpack_sum(pks, lvs, off, s, 1.0 / K)
    tol = 1e-5 * float(np.max(np.abs(want)))
    assert np.all(np.abs(got.astype(np.float64) - want) <= tol)
    db = DeviceBucket(np.zeros(total, np.float32), off)
    assert np.array_equal(got, db.unpack_sum(pks, lvs, s, 1.0 / K))
