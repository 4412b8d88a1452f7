"""Full-size parity on the ResNet-50- and VGG-19-shaped buckets, in the launch configuration the
benchmark times (same entry points, same grid sizing, K = 8 workers for the sum).

Where the oracle finishes in seconds the comparison is element by element; for the three large
VGG-19 FC weights the ORQ levels are checked through the discrete optimal condition itself, which
determines each level uniquely up to ties and holds at any size.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import ogq_workloads as wl
import paper_2002_11082_b200 as ogq

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_helpers import DeviceBucket

ORACLE_MAX = 5_000_000  # tensors up to this size get the element-by-element oracle


class SortedView:
    """The tensor sorted once (fp32 comparisons are exact) with fp64 prefix sums, so that the checks
    below cost a few binary searches per level whatever the tensor's size."""

    def __init__(self, v):
        self.sv = np.sort(v)
        self.cs = np.zeros(v.size + 1, np.float64)
        np.cumsum(self.sv, dtype=np.float64, out=self.cs[1:])

    def segment(self, L, R):
        """(count, sum) of {L <= v <= R} and the index range in the sorted array."""
        i0 = int(np.searchsorted(self.sv, L, side="left"))
        i1 = int(np.searchsorted(self.sv, R, side="right"))
        return i0, i1, self.cs[i1] - self.cs[i0]


def check_orq_levels_by_condition(v, lv, view=None):
    """Each level is a data value and satisfies, against the two levels it was solved from,
    count{b <= v <= R} >= T >= count{b < v <= R} with T = sum_{L<=v<=R}(v - L)/(R - L)
    (discrete form of the simplified optimal condition, applied in the order of Algorithm 1)."""
    view = view if view is not None else SortedView(v)
    s = lv.size
    assert lv[0] == view.sv[0] and lv[-1] == view.sv[-1]

    def rec(l, r):
        if r - l < 2:
            return
        m = (l + r) // 2
        L, R, b = lv[l], lv[r], lv[m]
        if R > L:
            i0, i1, ssum = view.segment(L, R)
            cnt = i1 - i0
            T = (ssum - float(L) * cnt) / (float(R) - float(L))
            ge = i1 - int(np.searchsorted(view.sv, b, side="left"))
            gt = i1 - int(np.searchsorted(view.sv, b, side="right"))
            assert ge > gt, "level is not a data value"
            slack = 1e-9 * cnt
            assert ge >= T - slack and gt <= T + slack, (l, r, ge, gt, T)
        else:
            assert b == L
        rec(l, m)
        rec(m, r)

    rec(0, s - 1)


def check_pb_level_by_condition(v, b1):
    """BinGrad-pb: g(b) = b n - sum_{|v| >= b} |v| is increasing in b and the level sits at its sign
    change (Eq. (bingrad-pb optimal condition) on magnitudes), so g is <= 0 one fp32 step below the
    level and >= 0 one step above it, up to the rounding of the fp64 sums."""
    a = np.abs(v)
    n = a.size
    b1 = np.float32(b1)
    lo, hi = np.nextafter(b1, np.float32(-np.inf)), np.nextafter(b1, np.float32(np.inf))

    def g(b):
        return float(b) * n - float(np.sum(a[a >= b], dtype=np.float64))

    tol = 1e-9 * n * float(b1) + 1e-300
    assert b1 >= 0 and g(lo) <= tol and g(hi) >= -tol, (b1, g(lo), g(hi))


def levels_close(got, want):
    tol = 1e-5 * float(np.max(np.abs(want)))
    return bool(np.all(np.abs(got.astype(np.float64) - want.astype(np.float64)) <= tol))


def worker_variants(db, K):
    """K simulated workers derived on the device from worker 0 (rolled and rescaled copies)."""
    g0 = db.grad
    return [g0 if k == 0 else (torch.roll(g0, 1001 * k) * (1.0 + 0.03 * k)).contiguous() for k in range(K)]


def run_bucket(bucket, orq_levels, with_bingrad_b, with_bingrad_pb=True):
    db = DeviceBucket(bucket.values, bucket.offsets)
    sizes = np.diff(bucket.offsets)
    if with_bingrad_pb:
        lv, _, st = db.levels_bingrad(ogq.OGQ_BINGRAD_PB, 0)
        assert not np.any(st & (ogq.OGQ_ST_INTERNAL | ogq.OGQ_ST_ITER_CAP | ogq.OGQ_ST_NONFINITE))
        for t in range(db.T):
            v = bucket.tensor(t)
            assert lv[t][0] == -lv[t][1]
            if sizes[t] <= ORACLE_MAX:
                want, _ = oracle.levels_bingrad_pb(v)
                assert levels_close(lv[t], want), (t, lv[t], want)
            else:
                check_pb_level_by_condition(v, lv[t][1])
        got, _ = db.quantize_pack(ogq.OGQ_BINGRAD_PB, 2, lv, None, 3, 2)
        want, _ = oracle.bucket_quantize_pack(bucket.values, bucket.offsets, oracle.PB, 2, lv, None, 3, 2)
        assert np.array_equal(got, want)
    for s in orq_levels:
        lv, st = db.levels_orq(s)
        assert not np.any(st & (ogq.OGQ_ST_INTERNAL | ogq.OGQ_ST_ITER_CAP | ogq.OGQ_ST_NONFINITE))
        exact = 0
        for t in range(db.T):
            v = bucket.tensor(t)
            if sizes[t] <= ORACLE_MAX:
                want, _ = oracle.levels_orq(v, s)
                assert levels_close(lv[t], want), (t, s, lv[t], want)
                exact += int(np.array_equal(lv[t], want))
            else:
                check_orq_levels_by_condition(v, lv[t])
                exact += 1
        assert exact >= db.T - 2
        # packed codes: bit-exact over the whole bucket, both sides on the same levels
        got, _ = db.quantize_pack(ogq.OGQ_ORQ, s, lv, None, 1, 0)
        want, _ = oracle.bucket_quantize_pack(bucket.values, bucket.offsets, oracle.ORQ, s, lv, None, 1, 0)
        assert np.array_equal(got, want)
    if with_bingrad_b:
        lv, th, st = db.levels_bingrad(ogq.OGQ_BINGRAD_B, 0)
        w_lv, w_th, w_st = oracle.bucket_levels_bingrad(bucket.values, bucket.offsets, oracle.B, 0)
        assert np.array_equal(st, w_st)
        for t in range(db.T):
            assert levels_close(lv[t], w_lv[t]) and abs(float(th[t]) - float(w_th[t])) <= 1e-5 * np.abs(w_lv[t]).max()
        got, _ = db.quantize_pack(ogq.OGQ_BINGRAD_B, 2, lv, th, 0, 0)
        want, _ = oracle.bucket_quantize_pack(bucket.values, bucket.offsets, oracle.B, 2, lv, th, 0, 0)
        assert np.array_equal(got, want)
    return db


def check_unpack_sum(db, s, K, full):
    """K = 8 workers quantized on the GPU, summed on the GPU, checked against the oracle's sum of
    the same packed buffers (whole bucket, or windows of the large tensors)."""
    bits = ogq.ogq_bits_for_levels(s)
    h_po = ogq.ogq_packed_layout(db.h_off, bits)
    po = torch.from_numpy(h_po).to(db.dev)
    grads = worker_variants(db, K)
    lvs, pks = [], []
    st = torch.zeros(db.T, dtype=torch.int32, device=db.dev)
    for k in range(K):
        lv = torch.zeros((db.T, s), device=db.dev)
        ogq.ogq_levels_orq(grads[k], db.off, db.T, db.N, s, lv, st, db.ws, db.ws_bytes)
        pk = torch.zeros(int(h_po[-1]), dtype=torch.int32, device=db.dev)
        ogq.ogq_quantize_pack(grads[k], db.off, db.T, db.N, ogq.OGQ_ORQ, s, lv, None, 5, k, po, pk)
        lvs.append(lv)
        pks.append(pk)
    out = torch.empty(db.N, device=db.dev)
    ogq.ogq_unpack_sum(ogq.device_pointer_array(pks), ogq.device_pointer_array(lvs), K, db.off, po, db.T, db.N, s,
                       1.0 / K, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    h_lv = [l.cpu().numpy() for l in lvs]
    h_pk = [p.cpu().numpy().view(np.uint32) for p in pks]
    sizes = np.diff(db.h_off)
    r = np.random.Generator(np.random.PCG64(99))
    for t in range(db.T):
        a, n = int(db.h_off[t]), int(sizes[t])
        if n == 0:
            continue
        region = [p[h_po[t] : h_po[t + 1]] for p in h_pk]
        lv_t = [l[t] for l in h_lv]
        if full or n <= ORACLE_MAX:
            want = oracle.unpack_sum(region, lv_t, n, bits, 1.0 / K)
            tol = 1e-5 * float(np.max(np.abs(want)))
            assert np.all(np.abs(got[a : a + n].astype(np.float64) - want) <= tol), t
        else:
            # windows that start on a 32-element boundary: their codes start on a word boundary
            starts = [0, (n - 70000) // 32 * 32] + [int(x) // 32 * 32 for x in r.integers(0, n - 70000, 6)]
            for e0 in starts:
                m = min(65536 + 37, n - e0)
                w0 = e0 * bits // 32
                sub = [p[w0 : w0 + (m * bits + 31) // 32 + 1] for p in region]
                want = oracle.unpack_sum(sub, lv_t, m, bits, 1.0 / K)
                tol = 1e-5 * float(np.max(np.abs(want)))
                assert np.all(np.abs(got[a + e0 : a + e0 + m].astype(np.float64) - want) <= tol), (t, e0)


def check_independent_workers(make_bucket, scheme, s, K):
    """K workers with independent data seeds: each worker's bucket is generated, quantized on the GPU
    and dropped again, only its levels and packed words are kept; then one unpack + sum over the K
    buffers.  Every worker's packed words and the whole dequantized sum are compared with the oracle."""
    b0 = make_bucket(0)
    db = DeviceBucket(b0.values, b0.offsets)
    bits = ogq.ogq_bits_for_levels(s)
    h_po = ogq.ogq_packed_layout(db.h_off, bits)
    po = torch.from_numpy(h_po).to(db.dev)
    lvs, pks = [], []
    for k in range(K):
        b = b0 if k == 0 else make_bucket(k)
        assert np.array_equal(b.offsets, b0.offsets)
        grad = db.grad if k == 0 else torch.from_numpy(b.values).to(db.dev)
        st = torch.zeros(db.T, dtype=torch.int32, device=db.dev)
        pk = torch.zeros(int(h_po[-1]), dtype=torch.int32, device=db.dev)
        if scheme == ogq.OGQ_ORQ:
            lv = torch.zeros((db.T, s), device=db.dev)
            ogq.ogq_levels_orq(grad, db.off, db.T, db.N, s, lv, st, db.ws, db.ws_bytes)
            ogq.ogq_quantize_pack(grad, db.off, db.T, db.N, scheme, s, lv, None, 5, k, po, pk)
            th = None
        else:
            lv = torch.zeros((db.T, 2), device=db.dev)
            th = torch.zeros(db.T, device=db.dev)
            ogq.ogq_levels_bingrad(grad, db.off, db.T, db.N, scheme, 0, lv, th, st, db.ws, db.ws_bytes)
            ogq.ogq_quantize_pack(grad, db.off, db.T, db.N, scheme, 2, lv, th, 5, k, po, pk)
        torch.cuda.synchronize()
        assert not np.any(st.cpu().numpy() & (ogq.OGQ_ST_INTERNAL | ogq.OGQ_ST_ITER_CAP | ogq.OGQ_ST_NONFINITE))
        h_lv = lv.cpu().numpy()
        h_th = th.cpu().numpy() if th is not None else None
        want, _ = oracle.bucket_quantize_pack(b.values, b.offsets, scheme, s, h_lv, h_th, 5, k)
        assert np.array_equal(pk.cpu().numpy().view(np.uint32), want), k
        if scheme == ogq.OGQ_BINGRAD_B:
            w_lv, w_th, _ = oracle.bucket_levels_bingrad(b.values, b.offsets, oracle.B, 0)
            for t in range(db.T):
                assert levels_close(h_lv[t], w_lv[t]), (k, t)
        lvs.append(lv)
        pks.append(pk)
        del grad, b
    out = torch.empty(db.N, device=db.dev)
    ogq.ogq_unpack_sum(ogq.device_pointer_array(pks), ogq.device_pointer_array(lvs), K, db.off, po, db.T, db.N, s,
                       1.0 / K, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    want = oracle.bucket_unpack_sum([p.cpu().numpy().view(np.uint32) for p in pks], [l.cpu().numpy() for l in lvs],
                                    db.h_off, s, 1.0 / K)
    for t in range(db.T):
        a, e = int(db.h_off[t]), int(db.h_off[t + 1])
        if e > a:
            tol = 1e-5 * float(np.max(np.abs(want[a:e])))
            assert np.all(np.abs(got[a:e].astype(np.float64) - want[a:e]) <= tol), t


def test_resnet50_bucket_full_size():
    b = wl.resnet50_bucket(0)
    assert b.num_tensors == 161 and b.total == 25557032
    db = run_bucket(b, orq_levels=(3, 9), with_bingrad_b=True)
    check_unpack_sum(db, 9, 8, full=True)
    check_unpack_sum(db, 3, 8, full=True)


@pytest.mark.parametrize("s", [3, 9])
def test_resnet50_eight_independent_workers(s):
    check_independent_workers(wl.resnet50_bucket, ogq.OGQ_ORQ, s, 8)


def test_vgg19_bucket_full_size():
    b = wl.vgg19_bucket(0)
    assert b.num_tensors == 38 and b.total == 143667240
    db = run_bucket(b, orq_levels=(9,), with_bingrad_b=True)
    check_unpack_sum(db, 9, 8, full=False)


def test_vgg19_bingrad_b_eight_independent_workers():
    check_independent_workers(wl.vgg19_bucket, ogq.OGQ_BINGRAD_B, 2, 8)


@pytest.mark.parametrize("log2n", [20, 24, 26, 28])
def test_flat_sweep_tensor(log2n):
    b = wl.sweep_tensor(log2n)
    db = DeviceBucket(b.values, b.offsets)
    view = SortedView(b.values) if b.total > ORACLE_MAX else None
    for s in (3, 5, 9, 17):
        lv, st = db.levels_orq(s)
        assert st[0] == 0
        if b.total <= ORACLE_MAX:
            want, _ = oracle.levels_orq(b.values, s)
            assert np.array_equal(lv[0], want)
        else:
            check_orq_levels_by_condition(b.values, lv[0], view)
        got, _ = db.quantize_pack(ogq.OGQ_ORQ, s, lv, None, 7, 1)
        want, _ = oracle.bucket_quantize_pack(b.values, b.offsets, oracle.ORQ, s, lv, None, 7, 1)
        assert np.array_equal(got, want)
    del view
    # BinGrad-b: levels, 1-bit codes, and the unpack of K = 1 worker (the dequantized gradient itself)
    lv, th, st = db.levels_bingrad(ogq.OGQ_BINGRAD_B, 0)
    w_lv, w_th, w_st = oracle.bucket_levels_bingrad(b.values, b.offsets, oracle.B, 0)
    assert st[0] == w_st[0] and levels_close(lv[0], w_lv[0])
    assert abs(float(th[0]) - float(w_th[0])) <= 1e-5 * float(np.abs(w_lv[0]).max())
    got, _ = db.quantize_pack(ogq.OGQ_BINGRAD_B, 2, lv, th, 0, 0)
    want, _ = oracle.bucket_quantize_pack(b.values, b.offsets, oracle.B, 2, lv, th, 0, 0)
    assert np.array_equal(got, want)
    out = db.unpack_sum([got], [lv], 2, 1.0)
    assert np.array_equal(out, oracle.bucket_unpack_sum([want], [lv], b.offsets, 2, 1.0))


def test_flat_tensor_with_crowded_cells():
    """A tensor large enough that every CTA streams more than 2^16 elements, 90 % of them one
    repeated non-zero value: the levels still satisfy the optimal condition exactly."""
    r = np.random.Generator(np.random.PCG64(23))
    n = 48_000_000
    v = wl.gaussian(r, n, 1e-3)
    v[r.random(n) < 0.9] = np.float32(2.5e-3)
    off = np.array([0, n], np.int64)
    db = DeviceBucket(v, off)
    for s in (3, 9):
        lv, st = db.levels_orq(s)
        assert st[0] == 0
        check_orq_levels_by_condition(v, lv[0])
    v[12_345_678] = np.nan
    db = DeviceBucket(v, off)
    lv, st = db.levels_orq(9)
    assert st[0] & ogq.OGQ_ST_NONFINITE


def test_resnet50_eight_workers_on_eight_streams():
    """The benchmark's launch configuration: K = 8 workers, each on a CUDA stream and a scratch buffer
    of its own, all in flight together.  Every worker's levels and packed words must equal what the
    same calls give one after the other on one stream (the kernels are bit-reproducible and share
    nothing between calls), and worker 0's levels must equal the oracle's."""
    K, s = 8, 9
    b = wl.resnet50_bucket(0)
    db = DeviceBucket(b.values, b.offsets)
    bits = ogq.ogq_bits_for_levels(s)
    h_po = ogq.ogq_packed_layout(db.h_off, bits)
    po = torch.from_numpy(h_po).to(db.dev)
    grads = worker_variants(db, K)

    def run(streams):
        lvs, pks, sts = [], [], []
        wss = [torch.empty(db.ws_bytes, dtype=torch.uint8, device=db.dev) for _ in range(K)]
        torch.cuda.synchronize()
        for k in range(K):
            lv = torch.zeros((db.T, s), device=db.dev)
            st = torch.zeros(db.T, dtype=torch.int32, device=db.dev)
            pk = torch.zeros(int(h_po[-1]), dtype=torch.int32, device=db.dev)
            lvs.append(lv); pks.append(pk); sts.append(st)
        torch.cuda.synchronize()
        for k in range(K):
            stream = streams[k] if streams else None
            ctx = torch.cuda.stream(stream) if stream is not None else torch.cuda.stream(torch.cuda.current_stream())
            with ctx:
                ogq.ogq_levels_orq(grads[k], db.off, db.T, db.N, s, lvs[k], sts[k], wss[k], db.ws_bytes, stream)
                ogq.ogq_quantize_pack(grads[k], db.off, db.T, db.N, ogq.OGQ_ORQ, s, lvs[k], None, 5, k, po, pks[k], stream)
        torch.cuda.synchronize()
        return [l.cpu().numpy() for l in lvs], [p.cpu().numpy() for p in pks], [x.cpu().numpy() for x in sts]

    serial = run(None)
    together = run([torch.cuda.Stream(device=db.dev) for _ in range(K)])
    for k in range(K):
        assert not np.any(together[2][k] & (ogq.OGQ_ST_INTERNAL | ogq.OGQ_ST_ITER_CAP | ogq.OGQ_ST_NONFINITE))
        assert np.array_equal(serial[0][k], together[0][k]), k
        assert np.array_equal(serial[1][k], together[1][k]), k
    want, _ = oracle.bucket_levels_orq(b.values, b.offsets, s)
    assert levels_close(together[0][0], want)


def test_orq_levels_when_the_rank_target_is_an_exact_integer():
    """A uniform grid of 17 values, each repeated 2^16 times (1.1 M elements): every T of Algorithm 1 is an
    integer up to fp64 rounding, so two neighbouring data values satisfy the discrete condition equally.
    The levels must be grid values that satisfy it (either choice), and the codes must match the oracle's
    for the levels returned."""
    reps = 1 << 16
    grid = (np.arange(17, dtype=np.float32) - 8.0) / np.float32(1024.0)
    v = np.repeat(grid, reps)
    np.random.Generator(np.random.PCG64(5)).shuffle(v)
    off = np.array([0, v.size], np.int64)
    db = DeviceBucket(v, off)
    view = SortedView(v)
    for s in (3, 5, 9, 17):
        lv, st = db.levels_orq(s)
        assert st[0] == 0 and np.all(np.isin(lv[0], grid))
        check_orq_levels_by_condition(v, lv[0], view)
        got, _ = db.quantize_pack(ogq.OGQ_ORQ, s, lv, None, 3, 0)
        want, _ = oracle.bucket_quantize_pack(v, off, oracle.ORQ, s, lv, None, 3, 0)
        assert np.array_equal(got, want)
