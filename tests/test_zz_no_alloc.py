"""The allocation-free gradient quantiser, `dqrm_grad_quant_int8_static`.

It exists for callers that cannot allocate device memory where they quantise (a plug-in
inside a framework that already owns the GPU's memory, or a loop that cannot take the
device-wide stall of cudaMalloc/cudaFree), so it has neither context nor workspace: its
scratch is a fixed array inside the library.  This file checks, through the C ABI, that
it gives the same scales and codes as `dqrm_grad_quant_int8`, and as the CPU oracle's
quantiser, on two calls in a row (the second with much smaller gradients, so maxima left
over from the first call would show),
and that a table count beyond the built-in limit is refused without launching anything.
It is collected last on purpose: a failure here leaves every other test already run.
"""
import numpy as np
import pytest

from dqrm_inputs import workloads as W

pytestmark = pytest.mark.gpu


def _sparse_grads(wl, step, scale):
    import oracle

    idx, off = W.make_batch(wl, step)
    go = (W.grad_out_np(wl, step) * np.float32(scale)).astype(np.float32)
    _, uniq_off, grad_rows = oracle.emb_bwd(go, wl.T, wl.D, wl.B, idx, off)
    return uniq_off, grad_rows


def test_static_quantiser_matches_workspace_quantiser_twice_in_a_row():
    import oracle
    import torch
    import paper_2410_20046_b200 as dq

    wl = W.scaled_down(W.kaggle(), total_rows=120_000, B=700, name="no_alloc_case")
    ctx = dq.Context(wl.row_off(), wl.D, wl.T * wl.B, wl.T * wl.B)
    for call, (step, scale) in enumerate([(0, 1.0), (1, 1e-3)]):
        uniq_off, grad_rows = _sparse_grads(wl, step, scale)
        U = grad_rows.shape[0]
        d_gr = torch.from_numpy(grad_rows).cuda()
        d_uo = torch.from_numpy(uniq_off).cuda()
        ref_codes = torch.empty((U, wl.D), dtype=torch.int8, device="cuda")
        ref_scales = torch.empty(wl.T, dtype=torch.float32, device="cuda")
        ctx.grad_quant_int8(d_gr, d_uo, ref_codes, ref_scales)
        ctx.raise_on_device_error()

        codes = torch.full((U, wl.D), 99, dtype=torch.int8, device="cuda")
        scales = torch.full((wl.T,), -1.0, dtype=torch.float32, device="cuda")
        rc = dq.grad_quant_int8_static(wl.T, wl.D, d_gr, d_uo, codes, scales)
        assert rc == dq.OK, f"call {call}: status {rc}"
        torch.cuda.synchronize()
        # integer codes and scales are compared bit for bit, as everywhere in this suite
        assert scales.cpu().numpy().tobytes() == ref_scales.cpu().numpy().tobytes(), f"call {call}: scales"
        assert torch.equal(codes, ref_codes), f"call {call}: codes"
        # ... and with the oracle's quantiser on the same host arrays
        o_codes, o_scales = oracle.grad_quant_int8(grad_rows, uniq_off, wl.D)
        assert scales.cpu().numpy().tobytes() == o_scales.tobytes(), f"call {call}: scales vs oracle"
        assert codes.cpu().numpy().tobytes() == o_codes.tobytes(), f"call {call}: codes vs oracle"
        assert int(codes.abs().max()) == 127
    ctx.close()


def test_static_quantiser_refuses_sizes_beyond_its_scratch():
    import torch
    import paper_2410_20046_b200 as dq

    T = dq.STATIC_MAX_TABLES + 1
    gr = torch.zeros((4, 16), dtype=torch.float32, device="cuda")
    uo = torch.zeros(T + 1, dtype=torch.int32, device="cuda")
    codes = torch.full((4, 16), 5, dtype=torch.int8, device="cuda")
    scales = torch.full((T,), -1.0, dtype=torch.float32, device="cuda")
    assert dq.grad_quant_int8_static(T, 16, gr, uo, codes, scales) == dq.ERR_STATIC_LIMIT
    torch.cuda.synchronize()
    assert int(codes.min()) == 5 and float(scales.max()) == -1.0      # nothing was written
    lib = dq.load_library()
    assert b"built-in scratch" in lib.dqrm_status_string(dq.ERR_STATIC_LIMIT)
