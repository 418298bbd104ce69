"""Host logic of the table-sharded step on CPU: the table plan, and two gloo ranks running the
whole step (indices to the owners, packed codes back, gradients to the owners, local update) with
the oracle as the compute, against the oracle's unsharded step on the full problem."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

from paper_2410_20046_b200.sharded import plan_tables


def test_plan_is_contiguous_complete_and_balanced():
    rows = [1000, 5, 7, 900, 20, 30, 40, 800, 3, 3, 3, 950]
    for world in (1, 2, 3, 4, 12):
        plan = plan_tables(rows, world)
        assert len(plan) == world and plan[0][0] == 0 and plan[-1][1] == len(rows)
        assert all(a[1] == b[0] for a, b in zip(plan, plan[1:])) and all(t1 > t0 for t0, t1 in plan)
    loads = [sum(rows[t0:t1]) for t0, t1 in plan_tables(rows, 4)]
    assert max(loads) <= 1.6 * sum(rows) / 4


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import sys
    import torch
    import torch.distributed as dist

    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    import oracle
    from paper_2410_20046_b200 import sharded
    from sharded_util import OracleShardCompute, problem

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B_local, bits = 24, 4
    wl, tables, idx2d, off, go = problem(world, B_local, bits=bits)
    plan = sharded.plan_tables(wl.rows, world)
    t0, t1 = plan[rank]
    ro = wl.row_off()
    compute = OracleShardCompute(oracle, tables[ro[t0]:ro[t1]].copy(), list(wl.rows[t0:t1]), wl.D, wl.B, bits, wl.lr)
    empty = lambda shape, dt: torch.empty(shape, dtype=getattr(torch, dt))
    step = sharded.TableShardedStep(compute, plan, rank, B_local, wl.D, bits, sharded.P2PExchange(), empty)
    step.refresh()
    mine = slice(rank * B_local, (rank + 1) * B_local)
    local_idx = torch.from_numpy(np.ascontiguousarray(idx2d[:, mine]))
    out = step.step(local_idx, lambda o: torch.from_numpy(np.ascontiguousarray(go[mine])))
    q.put((rank, out.numpy().copy(), compute.tables.copy(), (t0, t1)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_equal_the_unsharded_step(oracle):
    from sharded_util import problem, reference

    world, B_local, bits = 2, 24, 4
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=180) for _ in range(world)), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    wl, tables, idx2d, off, go = problem(world, B_local, bits=bits)
    want_out, want_tables = reference(oracle, wl, tables, idx2d, off, go, bits)
    ro = wl.row_off()
    for rank, out, local_tables, (t0, t1) in res:
        assert out.tobytes() == want_out[rank * B_local:(rank + 1) * B_local].tobytes()
        assert local_tables.tobytes() == want_tables[ro[t0]:ro[t1]].tobytes()
