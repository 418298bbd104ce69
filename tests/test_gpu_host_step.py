"""GPU parity of dqrm_train_step_host (host buffers in, pooled output back to the host, transfers on
streams of the context beside the kernels) against the oracle, over consecutive calls that reuse
the two sets of staging buffers in turn, with and without the overlap."""
import numpy as np
import pytest

from dqrm_inputs import workloads as W
from gpu_util import Case, assert_close_fp32, bit_equal

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("overlap", [True, False])
@pytest.mark.parametrize("name", ["kaggle_small", "multihot_small"])
def test_host_step_equals_oracle(oracle, name, overlap):
    import torch

    wl = {"kaggle_small": W.scaled_down(W.kaggle(), total_rows=300_000, B=2048, name="kaggle_small"),
          "multihot_small": W.scaled_down(W.multihot(), total_rows=26 * 3000, B=300, name="multihot_small")}[name]
    c = Case(wl, host_step=True)
    c.ctx.set_overlap(overlap)
    o_tables = W.tables_np(wl)
    d_tables = c.dev(o_tables)
    scales = c.empty(wl.T, torch.float32)
    c.ctx.scale_refresh(d_tables, c.bits, scales)
    torch.cuda.synchronize()
    o_scales, _ = oracle.scale_refresh(o_tables, c.row_off, wl.D, c.bits_np)
    steps = 6          # both staging sets are used three times
    batches = [c.batch(s) for s in range(steps)]
    pinned = [tuple(torch.from_numpy(np.ascontiguousarray(a)).pin_memory() for a in b) for b in batches]
    outs = [torch.full((wl.B, wl.T, wl.D), float("nan"), dtype=torch.float32).pin_memory() for _ in range(steps)]
    # all calls back to back, no host synchronisation in between: the staging buffers' reuse is ordered by the library
    for (idx, off, go), out in zip(pinned, outs):
        c.ctx.train_step_host(d_tables, idx, off, go, scales, c.bits, out, wl.lr, B=wl.B, L=len(idx))
    torch.cuda.current_stream().synchronize()     # the caller's stream alone: the copies must be complete behind it
    got = [o.numpy().copy() for o in outs]
    torch.cuda.synchronize()
    c.ctx.raise_on_device_error()
    for s, (idx, off, go) in enumerate(batches):
        r = oracle.train_step(o_tables, c.row_off, wl.D, wl.B, idx, off, go, o_scales, c.bits_np, wl.lr)
        assert_close_fp32(got[s], r["out"], f"step {s}: pooled output")
    assert bit_equal(d_tables.cpu().numpy(), o_tables)
    c.ctx.close()
