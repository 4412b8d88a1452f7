"""GPU parity: every stage of the CUDA path, called through the C ABI, against the CPU oracle
on the same seeded inputs.

Tolerances (also stated in the design notes):
  * levels: |gpu - oracle| <= 1e-5 * max_k |b_k| of the tensor (ORQ levels are data values, so
    they are normally bit-equal);
  * packed codes: bit-exact when both sides use the oracle's levels and the same Philox stream;
  * dequantized sums: |gpu - oracle| <= 1e-5 * max_i |out_i| of the tensor.
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

RAGGED_SIZES = [0, 1, 2, 3, 4, 5, 31, 32, 33, 127, 128, 129, 1000, 4097, 0, 70001, 262147, 7]


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def ragged_bucket(seed=5, sizes=RAGGED_SIZES):
    r = rng(seed)
    parts = []
    for i, n in enumerate(sizes):
        gen = [wl.laplace, wl.gaussian][i % 2]
        parts.append(gen(r, n, 10.0 ** r.uniform(-5, -2)) if n else np.zeros(0, np.float32))
    vals = np.concatenate(parts)
    return wl.Bucket(vals, wl.offsets_from_sizes(sizes), [str(n) for n in sizes])


def assert_levels_close(got, want, what=""):
    for t in range(want.shape[0]):
        tol = 1e-5 * float(np.max(np.abs(want[t]))) if want.shape[1] else 0.0
        assert np.all(np.abs(got[t].astype(np.float64) - want[t].astype(np.float64)) <= tol), (what, t, got[t], want[t])


# ------------------------------------------------------------------ BinGrad-b levels


@pytest.mark.parametrize("bucket_fn", [wl.config1, wl.config2, ragged_bucket])
@pytest.mark.parametrize("lloyd", [0, 3])
def test_levels_bingrad_b(bucket_fn, lloyd):
    b = bucket_fn()
    db = DeviceBucket(b.values, b.offsets)
    lv, th, st = db.levels_bingrad(ogq.OGQ_BINGRAD_B, lloyd)
    w_lv, w_th, w_st = oracle.bucket_levels_bingrad(b.values, b.offsets, oracle.B, lloyd)
    assert np.array_equal(st, w_st)
    assert_levels_close(lv, w_lv, "levels")
    for t in range(db.T):
        tol = 1e-5 * max(abs(float(w_lv[t, 0])), abs(float(w_lv[t, 1])))
        assert abs(float(th[t]) - float(w_th[t])) <= tol
    # run-to-run reproducibility (fixed reduction order)
    lv2, th2, _ = db.levels_bingrad(ogq.OGQ_BINGRAD_B, lloyd)
    assert np.array_equal(lv, lv2) and np.array_equal(th, th2)


def test_levels_bingrad_b_degenerate():
    vals = np.concatenate([np.full(1000, 0.5, np.float32), np.array([1.0], np.float32),
                           np.array([1.0, np.nan, 2.0, 3.0], np.float32)])
    off = np.array([0, 1000, 1001, 1005], np.int64)
    db = DeviceBucket(vals, off)
    lv, th, st = db.levels_bingrad(ogq.OGQ_BINGRAD_B, 0)
    assert st[0] & ogq.OGQ_ST_CONSTANT and lv[0, 0] == lv[0, 1] == th[0] == np.float32(0.5)
    assert st[1] & ogq.OGQ_ST_CONSTANT and lv[1, 0] == lv[1, 1] == 1.0
    assert st[2] & ogq.OGQ_ST_NONFINITE


# ------------------------------------------------------------------ ORQ and BinGrad-pb levels


def special_bucket(seed=9):
    """Distributions that stress the selection: zeros, duplicates, extreme scales, one-sided data,
    sizes around the shared-memory sort limit, constants and single elements."""
    r = rng(seed)
    parts = []
    z = wl.laplace(r, 100000, 1e-3); z[r.random(100000) < 0.6] = 0; parts.append(z)
    parts.append((np.round(wl.gaussian(r, 100000, 1e-3) * 3000) / 3000).astype(np.float32))
    parts.append(np.abs(wl.laplace(r, 50000, 1e-3)))
    parts.append((np.arange(100001) / 100000).astype(np.float32))
    parts.append(wl.laplace(r, 30000, 1e-30))
    parts.append(wl.laplace(r, 30000, 1e25))
    parts.append(wl.student_t(r, 4095, 3.0, 1e-3))
    parts.append(wl.student_t(r, 4096, 3.0, 1e-3))
    parts.append(wl.student_t(r, 4097, 3.0, 1e-3))
    parts.append(np.full(5000, -0.25, np.float32))
    parts.append(np.array([3.5], np.float32))
    parts.append(np.array([-1.0, 2.0], np.float32))
    parts.append(np.zeros(6000, np.float32))
    parts.append(-np.abs(wl.gaussian(r, 8191, 1e-2)))
    parts.append(np.concatenate([np.zeros(9000, np.float32), np.array([1.0, -1.0], np.float32)]))
    vals = np.concatenate(parts)
    return wl.Bucket(vals, wl.offsets_from_sizes([p.size for p in parts]), [str(i) for i in range(len(parts))])


def adversarial_bucket(seed=13):
    """Outliers, few distinct values, geometric ladders over many binades, shifted and two-cluster
    data: the cases where neighbouring order statistics sit in far-apart, sparsely filled cells."""
    r = rng(seed)
    parts = []
    for n in (5000, 17000, 60000):
        v = wl.gaussian(r, n, 1e-3)
        idx = r.integers(0, n, 25)
        v[idx] *= (10.0 ** r.uniform(1, 6, 25)).astype(np.float32)
        parts.append(v)
        vals = wl.gaussian(r, 5, 1e-2)
        parts.append(vals[r.integers(0, 5, n)])
        lad = (np.float32(3e-2) * np.float32(2.0) ** (-r.integers(0, 60, n)).astype(np.float32)).astype(np.float32)
        parts.append(lad * np.where(r.random(n) < 0.5, -1, 1).astype(np.float32))
        parts.append(wl.gaussian(r, n, 1e-4) + np.float32(0.37))
        parts.append(np.concatenate([wl.gaussian(r, n // 2, 1e-2), wl.gaussian(r, n - n // 2, 1e-6) + np.float32(0.5)]))
        parts.append(wl.student_t(r, n, 1.2, 1e-4))
    vals = np.concatenate(parts).astype(np.float32)
    return wl.Bucket(vals, wl.offsets_from_sizes([p.size for p in parts]), [str(i) for i in range(len(parts))])


@pytest.mark.parametrize("s", [3, 5, 9, 17])
@pytest.mark.parametrize("bucket_fn", [wl.config1, wl.config2, ragged_bucket, special_bucket, adversarial_bucket])
def test_levels_orq(bucket_fn, s):
    b = bucket_fn()
    db = DeviceBucket(b.values, b.offsets)
    lv, st = db.levels_orq(s)
    w_lv, w_st = oracle.bucket_levels_orq(b.values, b.offsets, s)
    assert np.array_equal(st, w_st), (st, w_st)
    assert_levels_close(lv, w_lv, "orq")
    # every level is one of the tensor's own values, so the match is normally bit-exact
    exact = sum(np.array_equal(lv[t], w_lv[t]) for t in range(db.T))
    assert exact >= db.T - 1
    lv2, _ = db.levels_orq(s)
    assert np.array_equal(lv, lv2)


@pytest.mark.parametrize("bucket_fn", [wl.config1, wl.config2, ragged_bucket, special_bucket, adversarial_bucket])
def test_levels_bingrad_pb(bucket_fn):
    b = bucket_fn()
    db = DeviceBucket(b.values, b.offsets)
    lv, _, st = db.levels_bingrad(ogq.OGQ_BINGRAD_PB)
    w_lv, _, w_st = oracle.bucket_levels_bingrad(b.values, b.offsets, oracle.PB)
    assert np.array_equal(st, w_st), (st, w_st)
    assert_levels_close(lv, w_lv, "pb")
    assert np.array_equal(lv[:, 0], -lv[:, 1])
    lv2, _, _ = db.levels_bingrad(ogq.OGQ_BINGRAD_PB)
    assert np.array_equal(lv, lv2)


def crowded_bucket(seed=17):
    """Tensors in which one non-zero value is repeated more than 2^16 times inside the piece a single
    CTA streams, next to ordinary data (the histogram's 32-bit partial sums must not wrap)."""
    r = rng(seed)
    parts = []
    for n, rep, frac in ((131072, 0.37, 0.95), (120000, -1.5e-3, 0.9), (131072, 2.5e-3, 0.7)):
        v = wl.gaussian(r, n, 1e-3)
        v[r.random(n) < frac] = np.float32(rep)
        parts.append(v)
    return wl.Bucket(np.concatenate(parts), wl.offsets_from_sizes([p.size for p in parts]), ["a", "b", "c"])


@pytest.mark.parametrize("s", [3, 9])
def test_levels_crowded_cells(s):
    b = crowded_bucket()
    db = DeviceBucket(b.values, b.offsets)
    lv, st = db.levels_orq(s)
    w_lv, w_st = oracle.bucket_levels_orq(b.values, b.offsets, s)
    assert np.array_equal(st, w_st)
    assert np.array_equal(lv, w_lv)
    lv, _, st = db.levels_bingrad(ogq.OGQ_BINGRAD_PB)
    w_lv, _, w_st = oracle.bucket_levels_bingrad(b.values, b.offsets, oracle.PB)
    assert np.array_equal(st, w_st)
    assert_levels_close(lv, w_lv, "pb")


def test_levels_nonfinite_is_flagged_not_trapped():
    vals = np.concatenate([wl.laplace(rng(1), 10000, 1e-3), wl.laplace(rng(2), 3000, 1e-3)])
    vals[77] = np.nan
    vals[10000 + 5] = np.inf
    off = np.array([0, 10000, 13000], np.int64)
    db = DeviceBucket(vals, off)
    lv, st = db.levels_orq(5)
    assert np.all(st & ogq.OGQ_ST_NONFINITE) and np.all(lv == 0)
    lv, _, st = db.levels_bingrad(ogq.OGQ_BINGRAD_PB)
    assert np.all(st & ogq.OGQ_ST_NONFINITE)


# ------------------------------------------------------------------ quantize + pack


@pytest.mark.parametrize("s", [3, 5, 9, 17])
@pytest.mark.parametrize("bucket_fn", [wl.config2, ragged_bucket])
def test_quantize_pack_orq_bit_exact(bucket_fn, s):
    b = bucket_fn()
    db = DeviceBucket(b.values, b.offsets)
    w_lv, _ = oracle.bucket_levels_orq(b.values, b.offsets, s)
    want, po = oracle.bucket_quantize_pack(b.values, b.offsets, oracle.ORQ, s, w_lv, None, 1, 3)
    got, g_po = db.quantize_pack(ogq.OGQ_ORQ, s, w_lv, None, 1, 3)
    assert np.array_equal(po, g_po)
    assert np.array_equal(got, want)
    other, _ = db.quantize_pack(ogq.OGQ_ORQ, s, w_lv, None, 1, 4)
    assert not np.array_equal(other, want)  # another stream id draws other numbers


@pytest.mark.parametrize("bucket_fn", [wl.config1, wl.config2, ragged_bucket])
def test_quantize_pack_bingrad_bit_exact(bucket_fn):
    b = bucket_fn()
    db = DeviceBucket(b.values, b.offsets)
    w_lv, w_th, _ = oracle.bucket_levels_bingrad(b.values, b.offsets, oracle.B, 0)
    want, _ = oracle.bucket_quantize_pack(b.values, b.offsets, oracle.B, 2, w_lv, w_th, 0, 0)
    got, _ = db.quantize_pack(ogq.OGQ_BINGRAD_B, 2, w_lv, w_th, 0, 0)
    assert np.array_equal(got, want)
    p_lv, _, _ = oracle.bucket_levels_bingrad(b.values, b.offsets, oracle.PB, 0)
    want, _ = oracle.bucket_quantize_pack(b.values, b.offsets, oracle.PB, 2, p_lv, None, (7 << 40) + 11, 2)
    got, _ = db.quantize_pack(ogq.OGQ_BINGRAD_PB, 2, p_lv, None, (7 << 40) + 11, 2)
    assert np.array_equal(got, want)


def test_quantize_special_values_and_duplicate_levels():
    lv = np.array([[0.0, 0.0, 0.0, 5.0, 5.0]], np.float32)
    vals = np.array([0.0, 5.0, 2.5, -1.0, 6.0, -0.0, np.nan, np.inf, -np.inf] * 57, np.float32)
    off = np.array([0, vals.size], np.int64)
    db = DeviceBucket(vals, off)
    want, _ = oracle.bucket_quantize_pack(vals, off, oracle.ORQ, 5, lv, None, 9, 1)
    got, _ = db.quantize_pack(ogq.OGQ_ORQ, 5, lv, None, 9, 1)
    assert np.array_equal(got, want)


# ------------------------------------------------------------------ unpack + sum


@pytest.mark.parametrize("s,K", [(2, 1), (3, 4), (5, 3), (9, 8), (17, 2), (9, 11), (9, 17), (3, 9), (2, 3)])
@pytest.mark.parametrize("bucket_fn", [wl.config2, ragged_bucket])
def test_unpack_sum(bucket_fn, s, K):
    base = bucket_fn()
    db = DeviceBucket(base.values, base.offsets)
    packed, levels = [], []
    for k in range(K):
        vals = base.values if k == 0 else (base.values * np.float32(1.0 + 0.1 * k)).astype(np.float32)
        if s == 2:
            lv, th, _ = oracle.bucket_levels_bingrad(vals, base.offsets, oracle.B, 0)
            pk, _ = oracle.bucket_quantize_pack(vals, base.offsets, oracle.B, 2, lv, th, 0, k)
        else:
            lv, _ = oracle.bucket_levels_orq(vals, base.offsets, s)
            pk, _ = oracle.bucket_quantize_pack(vals, base.offsets, oracle.ORQ, s, lv, None, 1, k)
        packed.append(pk)
        levels.append(lv)
    for scale in (1.0, 1.0 / K):
        want = oracle.bucket_unpack_sum(packed, levels, base.offsets, s, scale)
        got = db.unpack_sum(packed, levels, s, scale)
        for t in range(db.T):
            a, e = int(base.offsets[t]), int(base.offsets[t + 1])
            if e > a:
                tol = 1e-5 * float(np.max(np.abs(want[a:e])))
                assert np.all(np.abs(got[a:e].astype(np.float64) - want[a:e]) <= tol), (t, scale)
    if K == 1:
        assert np.array_equal(got, want)  # one worker: plain dequantization, exact


# ------------------------------------------------------------------ argument validation (no kernels run)


def test_argument_validation():
    b = wl.config1()
    db = DeviceBucket(b.values, b.offsets)
    lv = torch.zeros((1, 4), device=db.dev)
    st = torch.zeros(1, dtype=torch.int32, device=db.dev)
    with pytest.raises(ogq.OgqError) as e:
        ogq.ogq_levels_orq(db.grad, db.off, 1, db.N, 4, lv, st, db.ws, db.ws_bytes)
    assert e.value.code == 2
    with pytest.raises(ogq.OgqError) as e:
        ogq.ogq_levels_orq(db.grad, db.off, 1, db.N, 3, lv, st, db.ws, 16)
    assert e.value.code == 3
    with pytest.raises(ogq.OgqError) as e:
        ogq.ogq_levels_orq(db.grad.data_ptr() + 4, db.off, 1, db.N - 1, 3, lv, st, db.ws, db.ws_bytes)
    assert e.value.code == 1
    with pytest.raises(ogq.OgqError) as e:
        ogq.ogq_levels_bingrad(db.grad, db.off, 1, db.N, 7, 0, lv, lv, st, db.ws, db.ws_bytes)
    assert e.value.code == 2
    torch.cuda.synchronize()
