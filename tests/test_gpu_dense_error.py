"""Base-s (entropy-dense) packing and the quantization-error kernels against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import ogq_workloads as wl
import paper_2002_11082_b200 as ogq

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_helpers import DeviceBucket


def ragged_bucket(seed):
    r = np.random.Generator(np.random.PCG64(seed))
    sizes = [70_001, 0, 1, 19, 20, 21, 52, 4099, 262_147, 33, 1_000_003, 13, 7, 28, 560_000]
    parts = [wl.laplace(r, n, 10.0 ** r.uniform(-5, -2)) if n else np.zeros(0, np.float32) for n in sizes]
    return np.concatenate(parts), wl.offsets_from_sizes(sizes)


def dense_quantize(db, s, levels, seed, stream_id):
    h_po = ogq.ogq_dense_layout(db.h_off, s)
    po = torch.from_numpy(h_po).to(db.dev)
    pad = 64
    buf = torch.full((int(h_po[-1]) + 2 * pad,), 0x5A5A5A5A, dtype=torch.int32, device=db.dev)
    d_lv = torch.from_numpy(np.ascontiguousarray(levels, np.float32)).to(db.dev)
    ogq.ogq_quantize_pack_dense(db.grad, db.off, db.T, db.N, s, d_lv, seed, stream_id, po, buf[pad : pad + int(h_po[-1])])
    torch.cuda.synchronize()
    h = buf.cpu().numpy().view(np.uint32)
    assert np.all(h[:pad] == 0x5A5A5A5A) and np.all(h[pad + int(h_po[-1]) :] == 0x5A5A5A5A), "canary overwritten"
    return h[pad : pad + int(h_po[-1])].copy(), h_po


@pytest.mark.parametrize("s", [3, 5, 9, 17])
def test_dense_layout_pack_and_unpack(s):
    assert ogq.ogq_dense_digits(s) == oracle.dense_digits(s)
    vals, off = ragged_bucket(70 + s)
    db = DeviceBucket(vals, off)
    assert np.array_equal(ogq.ogq_dense_layout(off, s), oracle.dense_layout(off, s))
    lv, st = db.levels_orq(s)
    got, h_po = dense_quantize(db, s, lv, 21, 4)
    # same codes as the bit-packed quantizer (the oracle's), packed by the oracle's base-s packer
    _, _, codes = oracle.bucket_quantize_pack(vals, off, oracle.ORQ, s, lv, None, 21, 4, return_codes=True)
    want, w_po = oracle.bucket_pack_dense(codes, off, s)
    assert np.array_equal(h_po, w_po) and np.array_equal(got, want)
    # K workers: the same data quantized with different stream ids, summed
    K = 3
    pks = [got] + [dense_quantize(db, s, lv, 21, 10 + k)[0] for k in range(1, K)]
    d_pk = [torch.from_numpy(p.view(np.int32)).to(db.dev) for p in pks]
    d_lv = [torch.from_numpy(lv).to(db.dev) for _ in range(K)]
    po = torch.from_numpy(h_po).to(db.dev)
    pad = 64
    buf = torch.full((db.N + 2 * pad,), 12345.0, device=db.dev)
    ogq.ogq_unpack_sum_dense(ogq.device_pointer_array(d_pk), ogq.device_pointer_array(d_lv), K, db.off, po, db.T, db.N, s,
                             1.0 / K, buf[pad : pad + db.N])
    torch.cuda.synchronize()
    h = buf.cpu().numpy()
    assert np.all(h[:pad] == 12345.0) and np.all(h[pad + db.N :] == 12345.0)
    want_sum = oracle.bucket_unpack_sum_dense(pks, [lv] * K, off, s, 1.0 / K)
    out = h[pad : pad + db.N]
    for t in range(db.T):
        a, e = int(off[t]), int(off[t + 1])
        if e > a:
            tol = 1e-5 * float(np.max(np.abs(want_sum[a:e])))
            assert np.all(np.abs(out[a:e].astype(np.float64) - want_sum[a:e]) <= tol), t


def test_dense_on_an_unaligned_bucket_and_size_check():
    r = np.random.Generator(np.random.PCG64(77))
    sizes = [3, 1001, 2, 40_005]
    vals = wl.gaussian(r, sum(sizes), 1e-3)
    off = wl.offsets_from_sizes(sizes)
    db = DeviceBucket(vals, off)
    for s in (3, 9):
        lv, _ = db.levels_orq(s)
        got, _ = dense_quantize(db, s, lv, 5, 0)
        _, _, codes = oracle.bucket_quantize_pack(vals, off, oracle.ORQ, s, lv, None, 5, 0, return_codes=True)
        assert np.array_equal(got, oracle.bucket_pack_dense(codes, off, s)[0])
    with pytest.raises(ogq.OgqError):
        ogq.ogq_dense_layout(off, 4)
    # wire size: the reason for the format
    N = 25_557_032
    for s, ratio in ((3, 20), (5, 13), (9, 10), (17, 7)):
        words = int(ogq.ogq_dense_layout(np.array([0, N], np.int64), s)[-1])
        assert abs(32.0 * N / (32.0 * words) - ratio) < 0.01


def test_quantization_error_kernels():
    vals, off = ragged_bucket(81)
    db = DeviceBucket(vals, off)
    for s in (3, 9, 17):
        lv, _ = db.levels_orq(s)
        pk, h_po = db.quantize_pack(ogq.OGQ_ORQ, s, lv, None, 3, 1)
        d_lv = torch.from_numpy(lv).to(db.dev)
        d_pk = torch.from_numpy(pk.view(np.int32)).to(db.dev)
        po = torch.from_numpy(h_po).to(db.dev)
        err = torch.full((db.T,), -1.0, dtype=torch.float64, device=db.dev)
        exp = torch.full((db.T,), -1.0, dtype=torch.float64, device=db.dev)
        ogq.ogq_quant_error(db.grad, db.off, db.T, db.N, s, d_lv, po, d_pk, err)
        ogq.ogq_expected_error(db.grad, db.off, db.T, db.N, s, d_lv, exp)
        torch.cuda.synchronize()
        err, exp = err.cpu().numpy(), exp.cpu().numpy()
        _, _, codes = oracle.bucket_quantize_pack(vals, off, oracle.ORQ, s, lv, None, 3, 1, return_codes=True)
        for t in range(db.T):
            v = vals[off[t] : off[t + 1]]
            w_err = oracle.quant_error(v, lv[t], codes[t])
            w_exp = oracle.expected_error(v, lv[t]) if v.size else 0.0
            assert abs(err[t] - w_err) <= 1e-12 * max(w_err, 1e-300), (t, err[t], w_err)
            assert abs(exp[t] - w_exp) <= 1e-12 * max(w_exp, 1e-300), (t, exp[t], w_exp)
    # BinGrad-b (deterministic): the realised error of its 1-bit codes
    lv, th, _ = db.levels_bingrad(ogq.OGQ_BINGRAD_B, 0)
    pk, h_po = db.quantize_pack(ogq.OGQ_BINGRAD_B, 2, lv, th, 0, 0)
    err = torch.zeros((db.T,), dtype=torch.float64, device=db.dev)
    ogq.ogq_quant_error(db.grad, db.off, db.T, db.N, 2, torch.from_numpy(lv).to(db.dev), torch.from_numpy(h_po).to(db.dev),
                        torch.from_numpy(pk.view(np.int32)).to(db.dev), err)
    torch.cuda.synchronize()
    _, _, codes = oracle.bucket_quantize_pack(vals, off, oracle.B, 2, lv, th, 0, 0, return_codes=True)
    for t in range(db.T):
        w = oracle.quant_error(vals[off[t] : off[t + 1]], lv[t], codes[t])
        assert abs(float(err[t]) - w) <= 1e-12 * max(w, 1e-300)
