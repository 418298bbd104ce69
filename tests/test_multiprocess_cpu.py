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
