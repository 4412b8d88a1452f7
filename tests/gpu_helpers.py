"""Shared helpers of the GPU parity tests: device buffers and calls through the C ABI."""
from __future__ import annotations

import numpy as np
import torch

import paper_2002_11082_b200 as ogq


class DeviceBucket:
    """A bucket resident on cuda:0 plus the scratch the solvers need."""

    def __init__(self, values: np.ndarray, offsets: np.ndarray, max_levels: int = 17):
        self.dev = torch.device("cuda:0")
        self.h_values = np.ascontiguousarray(values, dtype=np.float32)
        self.h_off = np.ascontiguousarray(offsets, dtype=np.int64)
        self.T = self.h_off.size - 1
        self.N = int(self.h_off[-1])
        self.grad = torch.from_numpy(self.h_values).to(self.dev) if self.N else torch.zeros(4, device=self.dev)
        self.off = torch.from_numpy(self.h_off).to(self.dev)
        self.ws_bytes = ogq.ogq_workspace_bytes(self.T, self.N, max_levels)
        self.ws = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device=self.dev)
        # poison the scratch: the library must not rely on its contents
        self.ws.fill_(0xA5)

    def levels_bingrad(self, variant: int, lloyd_iters: int = 0):
        lv = torch.full((self.T, 2), float("nan"), device=self.dev)
        th = torch.full((self.T,), float("nan"), device=self.dev)
        st = torch.full((self.T,), -1, dtype=torch.int32, device=self.dev)
        ogq.ogq_levels_bingrad(self.grad, self.off, self.T, self.N, variant, lloyd_iters, lv, th, st,
                               self.ws, self.ws_bytes)
        torch.cuda.synchronize()
        return lv.cpu().numpy(), th.cpu().numpy(), st.cpu().numpy()

    def levels_orq(self, s: int):
        lv = torch.full((self.T, s), float("nan"), device=self.dev)
        st = torch.full((self.T,), -1, dtype=torch.int32, device=self.dev)
        ogq.ogq_levels_orq(self.grad, self.off, self.T, self.N, s, lv, st, self.ws, self.ws_bytes)
        torch.cuda.synchronize()
        return lv.cpu().numpy(), st.cpu().numpy()

    def quantize_pack(self, scheme: int, s: int, levels, thresh, seed: int, stream_id: int, tau=None):
        bits = ogq.ogq_bits_for_levels(s)
        h_po = ogq.ogq_packed_layout(self.h_off, bits)
        po = torch.from_numpy(h_po).to(self.dev)
        # canaries on both sides of the output
        pad = 64
        buf = torch.full((int(h_po[-1]) + 2 * pad,), 0x5A5A5A5A, dtype=torch.int32, device=self.dev)
        packed = buf[pad : pad + int(h_po[-1])]
        d_lv = torch.from_numpy(np.ascontiguousarray(levels, dtype=np.float32)).to(self.dev) if levels is not None else None
        d_th = torch.from_numpy(np.ascontiguousarray(thresh, dtype=np.float32)).to(self.dev) if thresh is not None else None
        if tau is None:
            ogq.ogq_quantize_pack(self.grad, self.off, self.T, self.N, scheme, s, d_lv, d_th, seed, stream_id, po, packed)
        else:
            ogq.ogq_quantize_pack_clipped(self.grad, self.off, self.T, self.N, scheme, s, d_lv, d_th, tau, seed,
                                          stream_id, po, packed)
        torch.cuda.synchronize()
        h = buf.cpu().numpy().view(np.uint32)
        assert np.all(h[:pad] == 0x5A5A5A5A) and np.all(h[pad + int(h_po[-1]) :] == 0x5A5A5A5A), "canary overwritten"
        return h[pad : pad + int(h_po[-1])].copy(), h_po

    def unpack_sum(self, packed_list, levels_list, s: int, scale: float):
        bits = ogq.ogq_bits_for_levels(s)
        h_po = ogq.ogq_packed_layout(self.h_off, bits)
        po = torch.from_numpy(h_po).to(self.dev)
        d_pk = [torch.from_numpy(np.ascontiguousarray(p).view(np.int32)).to(self.dev) if p.size else
                torch.zeros(4, dtype=torch.int32, device=self.dev) for p in packed_list]
        d_lv = [torch.from_numpy(np.ascontiguousarray(l, dtype=np.float32)).to(self.dev) for l in levels_list]
        pk_ptrs = ogq.device_pointer_array(d_pk)
        lv_ptrs = ogq.device_pointer_array(d_lv)
        pad = 64
        buf = torch.full((self.N + 2 * pad,), 12345.0, device=self.dev)
        out = buf[pad : pad + self.N]
        ogq.ogq_unpack_sum(pk_ptrs, lv_ptrs, len(d_pk), self.off, po, self.T, self.N, s, scale, out)
        torch.cuda.synchronize()
        h = buf.cpu().numpy()
        assert np.all(h[:pad] == 12345.0) and np.all(h[pad + self.N :] == 12345.0), "canary overwritten"
        return h[pad : pad + self.N].copy()
