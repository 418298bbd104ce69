"""GPU parity of the table-sharded step: W ranks emulated as host threads of one process on one GPU
(only the host threads wait on one another, at an in-memory exchange; no kernel waits on another),
every rank running the CUDA library on its own tables, against the oracle's unsharded step.
Also the two kernels on their own against the oracle."""
import threading

import numpy as np
import pytest

from dqrm_inputs import workloads as W
from gpu_util import Case, bit_equal
from sharded_util import problem, reference

pytestmark = pytest.mark.gpu


class LocalFabric:
    """In-process stand-in for the point-to-point exchange: a slot per rank and two barriers."""

    def __init__(self, world):
        self.world, self.slots, self.bar = world, [None] * world, threading.Barrier(world)

    def endpoint(self, rank):
        def exchange(send, recv_like):
            import torch

            torch.cuda.synchronize()
            self.slots[rank] = [s.contiguous() for s in send]
            self.bar.wait()
            got = [self.slots[r][rank].clone() for r in range(self.world)]
            torch.cuda.synchronize()
            self.bar.wait()
            return got
        return exchange


@pytest.mark.parametrize("world", [1, 2, 4])
@pytest.mark.parametrize("bits", [4, 8])
def test_sharded_step_equals_unsharded_oracle(oracle, world, bits):
    import torch
    from paper_2410_20046_b200 import sharded

    B_local = 96
    wl, tables, idx2d, off, go = problem(world, B_local, bits=bits)
    want_out, want_tables = reference(oracle, wl, tables, idx2d, off, go, bits)
    plan = sharded.plan_tables(wl.rows, world)
    ro = wl.row_off()
    fabric = LocalFabric(world)
    results, errors = [None] * world, []
    empty = lambda shape, dt: torch.empty(shape, dtype=getattr(torch, dt), device="cuda")

    def run(rank):
        try:
            torch.cuda.set_device(0)
            t0, t1 = plan[rank]
            c = sharded.GpuShardCompute(list(wl.rows[t0:t1]), wl.D, wl.B, bits, wl.lr)
            c.tables = torch.from_numpy(tables[ro[t0]:ro[t1]].copy()).cuda()
            step = sharded.TableShardedStep(c, plan, rank, B_local, wl.D, bits, fabric.endpoint(rank), empty)
            step.refresh()
            mine = slice(rank * B_local, (rank + 1) * B_local)
            out = step.step(torch.from_numpy(np.ascontiguousarray(idx2d[:, mine])).cuda(),
                            lambda o: torch.from_numpy(np.ascontiguousarray(go[mine])).cuda())
            torch.cuda.synchronize()
            c.ctx.raise_on_device_error()
            results[rank] = (out.cpu().numpy(), c.tables.cpu().numpy(), (t0, t1))
            c.ctx.close()
        except BaseException as e:          # noqa: BLE001  (reported by the main thread)
            errors.append(e)
            fabric.bar.abort()

    threads = [threading.Thread(target=run, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    for rank, (out, local_tables, (t0, t1)) in enumerate(results):
        assert bit_equal(out, want_out[rank * B_local:(rank + 1) * B_local])
        assert bit_equal(local_tables, want_tables[ro[t0]:ro[t1]])


@pytest.mark.parametrize("name,bits", [("kaggle_small", 4), ("terabyte_small", 4), ("kaggle_small", 2),
                                       ("terabyte_small", 8), ("odd_d20", 4), ("wide_d384", 8)])
def test_payload_kernels_against_oracle(oracle, name, bits):
    from dataclasses import replace

    wls = {
        "kaggle_small": W.scaled_down(W.kaggle(), total_rows=300_000, B=2048, name="kaggle_small"),
        "terabyte_small": W.scaled_down(W.terabyte(), total_rows=400_000, B=1500, name="terabyte_small"),
        "odd_d20": replace(W.scaled_down(W.kaggle(), total_rows=50_000, B=333), D=20, name="odd_d20"),
        "wide_d384": W.Workload("wide_d384", (700, 90, 5000), D=384, B=257, alpha=1.1, bits=8),
    }
    wl = wls[name]
    c = Case(wl)
    t = c.torch
    tables = W.tables_np(wl)
    b = np.full(wl.T, bits, dtype=np.int32)
    scales, _ = oracle.scale_refresh(tables, c.row_off, wl.D, b)
    idx, off, _ = c.batch(0)
    want = oracle.emb_fwd_codes(tables, c.row_off, wl.D, wl.B, idx, off, scales, bits)
    guard = 64
    payload = t.full((want.size + guard,), 0xA5, dtype=t.uint8, device="cuda")
    c.ctx.emb_fwd_codes(c.dev(tables), c.dev(idx), c.dev(off), c.dev(scales), bits, payload, B=wl.B, L=len(idx))
    c.ctx.raise_on_device_error()
    got = payload.cpu().numpy()
    assert (got[want.size:] == 0xA5).all()
    assert bit_equal(got[:want.size].reshape(want.shape), want)
    # decode two blocks of tables into one output; equals the training forward bit for bit
    out = t.full((wl.B, wl.T, wl.D), float("nan"), dtype=t.float32, device="cuda")
    cut = max(1, wl.T // 3)
    for t0, t1 in ((0, cut), (cut, wl.T)):
        if t1 > t0:
            blk = c.dev(np.ascontiguousarray(want[:, t0:t1, :]))
            c.ctx.decode_payload(blk, c.dev(scales[t0:t1]), bits, out, B=wl.B, T_blk=t1 - t0, T_total=wl.T, t0=t0)
    c.ctx.raise_on_device_error()
    fwd = oracle.emb_fwd(tables, c.row_off, wl.D, wl.B, idx, off, scales, b)
    assert bit_equal(out.cpu().numpy(), fwd)
    c.ctx.close()


def test_payload_call_refuses_multi_index_batches():
    import paper_2410_20046_b200 as dq

    wl = W.scaled_down(W.multihot(), total_rows=26 * 3000, B=64, name="mh")
    c = Case(wl)
    t = c.torch
    idx, off, _ = c.batch(0)
    with pytest.raises(dq.DqrmError):
        c.ctx.emb_fwd_codes(c.dev(W.tables_np(wl)), c.dev(idx), c.dev(off), c.empty(wl.T, t.float32), 4,
                            c.empty(wl.B * wl.T * wl.D // 2, t.uint8), B=wl.B, L=len(idx))
    c.ctx.close()
