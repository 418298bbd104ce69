"""World-size-2 checks of the benchmark's multi-process host logic on the gloo backend:
ranks take disjoint batches, and the job's time is the slowest rank's."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import torch.distributed as dist
    from dqrm_inputs import workloads as W
    from paper_2410_20046_b200 import harness

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = W.tiny()
    ids = [harness.batch_id(b, rank, world, 4) for b in range(4)]
    idx, _ = W.make_batch(wl, ids[0])
    ms = harness.max_over_ranks(10.0 + 5.0 * rank)
    q.put((rank, ids, idx[:8].tolist(), ms, harness.job_throughput(512, world, 10, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_disjoint_batches_and_time_is_max_over_ranks():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, ids0, idx0, ms0, v0), (r1, ids1, idx1, ms1, v1) = res
    assert not set(ids0) & set(ids1)
    assert idx0 != idx1                                  # different samples on each rank
    assert ms0 == ms1 == 15.0                            # the slowest rank's time, on every rank
    assert v0 == v1 == 512 * 2 * 10 / 15e-3              # all ranks' lookups over that time


def test_single_process_is_identity():
    from paper_2410_20046_b200 import harness

    assert harness.max_over_ranks(3.5) == 3.5
    assert harness.batch_id(3, 0, 1, 16) == 3


def _dp_worker(rank, world, port, q):
    import numpy as np
    import torch
    import torch.distributed as dist
    import oracle
    from dqrm_inputs import workloads as W
    from paper_2410_20046_b200 import dp

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = W.tiny()
    idx, off = W.make_batch(wl, 30 + rank)
    ur, uo, gr = oracle.emb_bwd(W.grad_out_np(wl, 30 + rank), wl.T, wl.D, wl.B, idx, off)
    # collective 1: unify the abs-max; then quantise locally (the oracle stands in for the CUDA call here)
    absmax = torch.from_numpy(oracle.grad_absmax(gr, uo, wl.D))
    dp.unify_absmax(absmax)
    scales = np.array([oracle.scale_from_absmax(a, 8) for a in absmax.numpy()], dtype=np.float32)
    codes = oracle.grad_quant_int8_scaled(gr, uo, wl.D, scales)
    # collective 2: gather every rank's rows and codes
    rows_cat, uoff_cat, codes_cat, stride, n, max_table = dp.gather_sparse(
        torch.from_numpy(ur), torch.from_numpy(uo), torch.from_numpy(codes))
    rows = [rows_cat[r, :int(uoff_cat[r, -1])].numpy() for r in range(world)]
    cds = [codes_cat[r, :int(uoff_cat[r, -1])].numpy() for r in range(world)]
    u_rows, u_off, sums = oracle.dp_merge(rows, [uoff_cat[r].numpy() for r in range(world)], cds, wl.T, wl.D)
    tables = W.tables_np(wl)
    oracle.row_update_i32(tables, wl.row_off(), wl.D, u_rows, u_off, sums, scales, wl.lr)
    q.put((rank, scales.tobytes(), tables.tobytes(), n, stride, max_table))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_gradient_exchange_keeps_replicas_identical_and_equals_one_process():
    import numpy as np
    import oracle
    from dqrm_inputs import workloads as W

    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_dp_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # what one process computes for the same two ranks
    wl = W.tiny()
    local = []
    for r in range(world):
        idx, off = W.make_batch(wl, 30 + r)
        local.append(oracle.emb_bwd(W.grad_out_np(wl, 30 + r), wl.T, wl.D, wl.B, idx, off))
    tables = W.tables_np(wl)
    want = oracle.dp_exchange_update(tables, wl.row_off(), wl.D, local, wl.lr)
    for rank, scales, tab, n, stride, max_table in res:
        assert scales == want["scales"].tobytes()
        assert tab == tables.tobytes()                        # both replicas equal the single-process result
        assert n == sum(len(l[0]) for l in local) and stride == max(len(l[0]) for l in local)
        assert max_table == max(sum(l[1][t + 1] - l[1][t] for l in local) for t in range(wl.T))
