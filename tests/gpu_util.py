"""Helpers of the GPU parity tests: run the CUDA library and the CPU oracle on the same
seeded inputs.  The oracle side never sees a value produced by the CUDA side."""
from __future__ import annotations

import numpy as np

from dqrm_inputs import workloads as W


class Case:
    """Host inputs of one workload (tables + per-step batches) and a CUDA context."""

    def __init__(self, wl, max_lookups=None, host_step=False, bits=None):
        import torch
        import paper_2410_20046_b200 as dq

        self.wl = wl
        self.torch = torch
        self.row_off = wl.row_off()
        self.samplers = W.make_samplers(wl)
        self.bits_np = np.full(wl.T, wl.bits, dtype=np.int32) if bits is None else np.asarray(bits, dtype=np.int32)
        self.G = wl.T * wl.B
        if max_lookups is None:
            max_lookups = self.G * (wl.bag_max if wl.bag_mean else 1)
        self.max_lookups = max_lookups
        self.ctx = dq.Context(self.row_off, wl.D, max_lookups, self.G, host_step=host_step)
        self.bits = torch.from_numpy(self.bits_np).cuda()

    def batch(self, step):
        idx, off = W.make_batch(self.wl, step, self.samplers)
        return idx, off, W.grad_out_np(self.wl, step)

    def dev(self, a):
        return self.torch.from_numpy(np.ascontiguousarray(a)).cuda()

    def empty(self, shape, dtype):
        return self.torch.empty(shape, dtype=dtype, device="cuda")

    # ---- single calls on given host inputs; return host arrays ----
    def gpu_refresh(self, d_tables):
        t = self.torch
        scales = self.empty(self.wl.T, t.float32)
        minmax = self.empty((self.wl.T, 2), t.float32)
        self.ctx.scale_refresh(d_tables, self.bits, scales, minmax)
        self.ctx.raise_on_device_error()
        return scales, minmax

    def gpu_fwd(self, d_tables, idx, off, d_scales, want_codes=True):
        t = self.torch
        L = len(idx)
        out = self.empty((self.wl.B, self.wl.T, self.wl.D), t.float32)
        codes = self.empty((max(L, 1), self.wl.D), t.int8) if want_codes else None
        self.ctx.emb_fwd(d_tables, self.dev(idx) if L else self.empty(1, t.int32), self.dev(off), d_scales,
                         self.bits, out, codes, B=self.wl.B, L=L)
        self.ctx.raise_on_device_error()
        return out.cpu().numpy(), (codes.cpu().numpy()[:L] if want_codes else None)

    def gpu_bwd(self, idx, off, grad_out):
        t = self.torch
        L = len(idx)
        ur = t.full((max(L, 1),), -7, dtype=t.int32, device="cuda")
        uo = self.empty(self.wl.T + 1, t.int32)
        gr = t.full((max(L, 1), self.wl.D), float("nan"), dtype=t.float32, device="cuda")
        self.ctx.emb_bwd(self.dev(grad_out), self.dev(idx) if L else self.empty(1, t.int32), self.dev(off),
                         ur, uo, gr, B=self.wl.B, L=L)
        self.ctx.raise_on_device_error()
        uo_h = uo.cpu().numpy()
        U = int(uo_h[-1])
        ur_h, gr_h = ur.cpu().numpy(), gr.cpu().numpy()
        # nothing at or beyond U is written
        assert (ur_h[U:] == -7).all() and np.isnan(gr_h[U:]).all()
        return ur_h[:U].copy(), uo_h, gr_h[:U].copy()

    def gpu_quant(self, grad_rows, uniq_off):
        t = self.torch
        U = grad_rows.shape[0]
        codes = self.empty((max(U, 1), self.wl.D), t.int8)
        gs = self.empty(self.wl.T, t.float32)
        self.ctx.grad_quant_int8(self.dev(grad_rows) if U else self.empty((1, self.wl.D), t.float32),
                                 self.dev(uniq_off), codes, gs)
        self.ctx.raise_on_device_error()
        return codes.cpu().numpy()[:U], gs.cpu().numpy()

    def gpu_update(self, d_tables, unique_rows, uniq_off, codes, grad_scales, lr):
        t = self.torch
        U = len(unique_rows)
        self.ctx.row_update(d_tables, self.dev(unique_rows) if U else self.empty(1, t.int32), self.dev(uniq_off),
                            self.dev(codes) if U else self.empty((1, self.wl.D), t.int8), self.dev(grad_scales), lr)
        self.ctx.raise_on_device_error()


def assert_close_fp32(got, want, what=""):
    """Tolerance of the FP32 outputs whose summation order may differ: 1e-5 relative,
    1e-6 absolute."""
    np.testing.assert_allclose(got, want, rtol=1e-5, atol=1e-6, err_msg=what)


def bit_equal(a, b):
    return a.shape == b.shape and a.tobytes() == b.tobytes()
