"""Gradient clipping fused into the level solvers, against the oracle's clip-then-solve.

tau = c * sigma is compared with the oracle's (two-pass, long double) value; everything after it
uses the threshold the GPU returned on both sides, because the clipped gradient, the levels and the
codes are exact functions of tau.
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
    from test_gpu_buckets import bucket_offsets, run_encode, close


def clip_bucket():
    r = np.random.Generator(np.random.PCG64(60))
    sizes = [300_001, 5, 0, 4096, 70_000, 1_500_000, 131_073, 1, 2_100_000]
    parts = []
    for i, n in enumerate(sizes):
        v = wl.student_t(r, n, 3.0, 10.0 ** r.uniform(-4, -2)) if n else np.zeros(0, np.float32)
        if i == 4:
            v = v + np.float32(3e-3)  # a mean far from zero: sigma is about the mean
        parts.append(v.astype(np.float32))
    return np.concatenate(parts), wl.offsets_from_sizes(sizes)


def gpu_tau(db, c):
    tau = torch.full((db.T,), float("nan"), device=db.dev)
    st = torch.full((db.T,), -1, dtype=torch.int32, device=db.dev)
    ogq.ogq_clip_threshold(db.grad, db.off, db.T, db.N, c, tau, st, db.ws, db.ws_bytes)
    torch.cuda.synchronize()
    return tau, st.cpu().numpy()


@pytest.mark.parametrize("c", [2.5, 1.7])
def test_clip_threshold_and_clipped_levels_and_codes(c):
    vals, off = clip_bucket()
    db = DeviceBucket(vals, off)
    d_tau, st = gpu_tau(db, c)
    tau = d_tau.cpu().numpy()
    w_tau, w_st = oracle.bucket_clip_thresholds(vals, off, c)
    assert np.array_equal(st, w_st)
    assert np.all(np.abs(tau.astype(np.float64) - w_tau) <= 1e-6 * np.abs(w_tau))
    clipped = oracle.bucket_clip(vals, off, tau)
    assert np.any(clipped != vals)

    for s in (3, 9):
        lv = torch.full((db.T, s), float("nan"), device=db.dev)
        stl = torch.full((db.T,), -1, dtype=torch.int32, device=db.dev)
        ogq.ogq_levels_orq_clipped(db.grad, db.off, db.T, db.N, s, d_tau, lv, stl, db.ws, db.ws_bytes)
        torch.cuda.synchronize()
        lv = lv.cpu().numpy()
        w_lv, w_stl = oracle.bucket_levels_orq(clipped, off, s)
        assert np.array_equal(stl.cpu().numpy(), w_stl)
        for t in range(db.T):
            assert close(lv[t], w_lv[t]), (t, s, lv[t], w_lv[t])
            if off[t + 1] - off[t] > 1 and tau[t] > 0 and np.abs(vals[off[t] : off[t + 1]]).max() > tau[t]:
                assert max(abs(lv[t][0]), abs(lv[t][-1])) == tau[t]  # Corollary 1 on the clipped gradient
        # the clamping quantizer on the raw gradient = the oracle's quantizer on the clipped gradient
        got, _ = db.quantize_pack(ogq.OGQ_ORQ, s, lv, None, 11, 2, tau=d_tau)
        want, _ = oracle.bucket_quantize_pack(clipped, off, oracle.ORQ, s, lv, None, 11, 2)
        assert np.array_equal(got, want)
        # the plain quantizer with the clipped levels may pick another of several equal end levels
        # for a value beyond tau, but decodes to the same values
        plain, _ = db.quantize_pack(ogq.OGQ_ORQ, s, lv, None, 11, 2)
        assert np.array_equal(oracle.bucket_unpack_sum([plain], [lv], off, s, 1.0),
                              oracle.bucket_unpack_sum([want], [lv], off, s, 1.0))

    for variant, o_variant in ((ogq.OGQ_BINGRAD_B, oracle.B), (ogq.OGQ_BINGRAD_PB, oracle.PB)):
        lv = torch.full((db.T, 2), float("nan"), device=db.dev)
        th = torch.full((db.T,), float("nan"), device=db.dev)
        stl = torch.full((db.T,), -1, dtype=torch.int32, device=db.dev)
        ogq.ogq_levels_bingrad_clipped(db.grad, db.off, db.T, db.N, variant, 0, d_tau, lv, th, stl, db.ws, db.ws_bytes)
        torch.cuda.synchronize()
        lv, th = lv.cpu().numpy(), th.cpu().numpy()
        w_lv, w_th, w_stl = oracle.bucket_levels_bingrad(clipped, off, o_variant, 0)
        assert np.array_equal(stl.cpu().numpy(), w_stl)
        for t in range(db.T):
            assert close(lv[t], w_lv[t]), (t, variant, lv[t], w_lv[t])
        th_in = th if variant == ogq.OGQ_BINGRAD_B else None
        got, _ = db.quantize_pack(variant, 2, lv, th_in, 11, 2, tau=d_tau)
        want, _ = oracle.bucket_quantize_pack(clipped, off, o_variant, 2, lv, th_in, 11, 2)
        assert np.array_equal(got, want)


def test_clip_threshold_reports_non_finite_values_and_large_tensors():
    b = wl.sweep_tensor(24)
    v = b.values.copy()
    db = DeviceBucket(v, b.offsets)
    d_tau, st = gpu_tau(db, 2.5)
    w_tau, _ = oracle.clip_threshold(v, 2.5)
    assert st[0] == 0 and abs(float(d_tau[0]) - float(w_tau)) <= 1e-6 * float(w_tau)
    v[123_456] = np.nan
    db = DeviceBucket(v, b.offsets)
    d_tau, st = gpu_tau(db, 2.5)
    assert st[0] == ogq.OGQ_ST_NONFINITE and float(d_tau[0]) == 0.0


def test_bucket_mode_with_clipping_is_the_imagenet_setting():
    """d = 512, c = 2.5 (the paper's distributed runs): per-bucket tau inside the fused kernel."""
    v = wl.resnet50_bucket(0).values[11_000_000:12_000_000 + 300]
    d, c = 512, 2.5
    off = bucket_offsets(v.size, d)
    w_tau, _ = oracle.bucket_clip_thresholds(v, off, c)
    clipped = oracle.bucket_clip(v, off, w_tau)
    for scheme, o_scheme, s in ((ogq.OGQ_ORQ, oracle.ORQ, 3), (ogq.OGQ_ORQ, oracle.ORQ, 9), (ogq.OGQ_BINGRAD_B, oracle.B, 2),
                                (ogq.OGQ_BINGRAD_PB, oracle.PB, 2)):
        lv, th, st, packed = run_encode(v, d, scheme, s, 0, seed=13, stream_id=1, clip_c=c)
        if scheme == ogq.OGQ_ORQ:
            w_lv, _ = oracle.bucket_levels_orq(clipped, off, s)
        else:
            w_lv, w_th, _ = oracle.bucket_levels_bingrad(clipped, off, o_scheme, 0)
        # tau is recomputed inside the kernel (fp64, other summation order): where its fp32 rounding
        # differs from the oracle's by an ulp the clipped extremes differ by that ulp too
        bad = [j for j in range(off.size - 1) if not close(lv[j], w_lv[j])]
        assert len(bad) == 0, bad[:5]
        # codes: both sides on the GPU's levels; a clipped value takes the code of +-tau either way
        th_in = th if scheme == ogq.OGQ_BINGRAD_B else None
        want, _ = oracle.bucket_quantize_pack(clipped, off, o_scheme, s, lv, th_in, 13, 1)
        assert np.array_equal(packed, want)
