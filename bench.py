#!/usr/bin/env python
"""Benchmark of the QAT embedding step (forward + backward + INT8 gradient quantisation +
touched-row update, scale refresh every `period` steps) on synthetic Criteo-shaped data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints ONE JSON line.  `value` is whole-job lookups/s with inputs resident in HBM,
`e2e` the same through the host-buffer entry point (copies inside the timed region),
`roofline` the dominant kernel against the measured HBM copy rate, `cpu_baseline` the
CPU oracle timed on the host cores.  With --impl reference the oracle itself is timed.
The default run (N = 1, workload kaggle_b16384) also measures terabyte_b32768 in the same
process and carries it in the line's `also` block.  With --gpus N > 1 and no launcher in
the environment the script starts N ranks itself (one process per GPU, torchrun).
By default consecutive steps are software-pipelined: the index sort of batch k+1 runs on a
second stream while batch k trains (--no-pipeline: one call per step).  --packed times the
bit-packed export and the packed inference lookup instead of the training step.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "QAT embedding lookups/sec (fwd+bwd+update)"
UNIT = "lookups/s"
N_BATCHES = 20
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def get_workload(name):
    from dqrm_inputs import workloads as W

    if name in W.BY_NAME:
        return W.BY_NAME[name]()
    if name.startswith("sweep_"):   # sweep_d64_b8_zipf: one table of 10 M rows, batch 65536 (feature size, bits, index law)
        try:
            d, b, dist = name.split("_")[1:]
            assert d[0] == "d" and b[0] == "b" and dist in ("uniform", "zipf")
            return W.sweep(D=int(d[1:]), bits=int(b[1:]), zipf=(dist == "zipf"))
        except (ValueError, AssertionError):
            raise SystemExit(f"bad sweep name {name}; expected sweep_d<16|32|64|128>_b<2|4|8>_<uniform|zipf>")
    if name == "terabyte_2gb_b32768":   # the Terabyte-shaped step over 2 GB of tables: small enough for a counter capture
        return W.scaled_down(W.terabyte(32768), total_rows=8_000_000, B=32768, name="terabyte_2gb_b32768")
    if name == "kaggle_smoke":      # small stand-in used by the tests of this script
        return W.scaled_down(W.kaggle(), total_rows=200_000, B=1024, name="kaggle_smoke")
    raise SystemExit(f"unknown workload {name}; choose from {sorted(W.BY_NAME)}")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def algorithmic_bytes(wl, L, G, U):
    """Bytes the method must move per call (each touched row once).  `step` counts what the calls of
    the fused step move; `step_separate_calls` adds the D*U bytes of INT8 codes that a separate update
    call reads back (8L + 8G + 8DG + U(8 + 22D))."""
    D = wl.D
    fwd = 4 * L + 4 * G + 4 * D * U + 4 * D * G
    bwd = 4 * D * G + 4 * L + 4 * G + 4 * U + 4 * D * U
    qu = 4 * D * U + D * U + 4 * U + 8 * D * U          # read grads, write codes, read rows, RMW rows
    return {"fwd": fwd, "bwd": bwd, "quant_update": qu, "step": fwd + bwd + qu,
            "step_separate_calls": 8 * L + 8 * G + 8 * D * G + U * (8 + 22 * D),
            "refresh": wl.table_bytes()}


def base_config(wl):
    """The workload, in the same words for both arms."""
    return {"workload": wl.name, "tables": wl.T, "dim": wl.D, "batch_per_gpu": wl.B, "bits": wl.bits, "grad_bits": 8,
            "refresh_period": wl.period, "table_bytes": wl.table_bytes(),
            "inputs": f"seeded synthetic batches, distinct per step and cycled ({N_BATCHES} on the GPU arm, 4 on the "
                      "CPU arm); one batch's rows, gradients and outputs plus the tables exceed the 126 MB L2"}


# kernel -> which algorithmic byte count bounds it (the sort kernels carry no algorithmic
# bytes of their own: they are implementation cost of the backward)
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (set an entry to None when its kernel has changed since the capture)
NCU_TRAFFIC = {
    ("kaggle_b16384", "seg_reduce_kernel"): 31.13e6,
    ("kaggle_b16384", "fwd_kernel"): 26.33e6,
    ("kaggle_b16384", "row_stream_kernel<fused>"): 25.25e6,
    # the Terabyte-shaped step captured over 2 GB of tables (the full tables are too large for a counter capture)
    ("terabyte_2gb_b32768", "seg_reduce_kernel"): 240.27e6,
    ("terabyte_2gb_b32768", "fwd_kernel"): 212.28e6,
    ("terabyte_2gb_b32768", "row_stream_kernel<fused>"): 79.73e6,
    # ... and scaled to the full tables by the reduce's algorithmic bytes (265.79 MB against 254.88 MB per launch):
    # its traffic is the upstream-gradient rows (the same) plus the unique rows it writes
    ("terabyte_b32768", "seg_reduce_kernel"): 250.55e6,
}

KERNEL_BYTES = {
    "fwd_kernel": lambda ab, wl, L, G, U: ab["fwd"],
    "seg_reduce_kernel": lambda ab, wl, L, G, U: 4 * wl.D * G + 4 * wl.D * U,
    "row_stream_kernel<fused>": lambda ab, wl, L, G, U: ab["quant_update"],
    "refresh_kernel": lambda ab, wl, L, G, U: ab["refresh"],
}


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def cpu_sample_steps(wl):
    """Steps of the CPU oracle that make about ten seconds of one-core work: the oracle does about 3.5 M lookups
    per second at 16 features per row, and its time per lookup grows with the row length."""
    per_step_s = wl.T * wl.B * max(1, wl.bag_mean or 1) / 3.5e6 * max(1.0, wl.D / 16)
    return int(min(100, max(3, round(10.0 / per_step_s))))


def oracle_sample(wl, tables_h, n_steps, period):
    """Times the CPU oracle, as it stands, on `n_steps` full batches and one refresh: on one host core,
    and on all cores of the affinity mask with one table per thread (tables are independent, so the
    results are the same bits; a single table splits nothing)."""
    import numpy as np
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    from dqrm_inputs import workloads as W

    off = wl.row_off()
    bits = np.full(wl.T, wl.bits, dtype=np.int32)
    samplers = W.make_samplers(wl)
    t0 = time.perf_counter()
    scales, _ = oracle.scale_refresh(tables_h, off, wl.D, bits)
    t_refresh = time.perf_counter() - t0
    distinct = [(*W.make_batch(wl, s, samplers), W.grad_out_np(wl, s)) for s in range(min(n_steps, 4))]
    batches = [distinct[s % len(distinct)] for s in range(n_steps)]      # cycled
    t_steps, lookups = 0.0, 0
    for idx, offs, go in batches:
        t0 = time.perf_counter()
        oracle.train_step(tables_h, off, wl.D, wl.B, idx, offs, go, scales, bits, wl.lr)
        t_steps += time.perf_counter() - t0
        lookups += len(idx)
    per_step = t_steps / n_steps + t_refresh / period
    one = ((lookups / n_steps) / per_step, t_steps / n_steps, t_refresh)

    # all cores: the same calls on one-table problems, a thread each (the C calls release the interpreter lock)
    cores = host_cores()
    threads = max(1, min(cores, wl.T))
    one_off = lambda t: np.array([0, off[t + 1] - off[t]], dtype=np.int64)

    def table_refresh(t):
        return oracle.scale_refresh(tables_h[off[t]:off[t + 1]], one_off(t), wl.D, bits[t:t + 1])

    def table_step(job):
        t, idx_t, offs_t, go_t = job
        oracle.train_step(tables_h[off[t]:off[t + 1]], one_off(t), wl.D, wl.B, idx_t, offs_t, go_t, scales[t:t + 1],
                          bits[t:t + 1], wl.lr)

    with ThreadPoolExecutor(max_workers=threads) as pool:
        t0 = time.perf_counter()
        list(pool.map(table_refresh, range(wl.T)))
        t_refresh_mc = time.perf_counter() - t0
        t_steps_mc = 0.0
        for idx, offs, go in batches:
            jobs = []
            for t in range(wl.T):                      # slicing the batch by table is the harness's work, not timed
                lo, hi = offs[t * wl.B], offs[(t + 1) * wl.B]
                jobs.append((t, np.ascontiguousarray(idx[lo:hi]),
                             np.ascontiguousarray(offs[t * wl.B:(t + 1) * wl.B + 1] - lo),
                             np.ascontiguousarray(go[:, t:t + 1, :])))
            t0 = time.perf_counter()
            list(pool.map(table_step, jobs))
            t_steps_mc += time.perf_counter() - t0
    per_step_mc = t_steps_mc / n_steps + t_refresh_mc / period
    many = ((lookups / n_steps) / per_step_mc, t_steps_mc / n_steps, t_refresh_mc, threads, cores)
    return one, many


def host_tables(wl):
    import torch
    from dqrm_inputs import workloads as W

    dev = "cuda" if torch.cuda.is_available() else "cpu"
    return W.tables_torch(wl, dev).cpu().numpy()


def run_reference(args):
    """The oracle on the host cores, timed step by step (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np
    import oracle
    from dqrm_inputs import workloads as W

    oracle.build()
    wl = get_workload(args.workload)
    tables_h = host_tables(wl)
    off = wl.row_off()
    bits = np.full(wl.T, wl.bits, dtype=np.int32)
    samplers = W.make_samplers(wl)
    t0 = time.perf_counter()
    scales, _ = oracle.scale_refresh(tables_h, off, wl.D, bits)
    t_refresh = time.perf_counter() - t0
    batches = [(*W.make_batch(wl, s, samplers), W.grad_out_np(wl, s)) for s in range(min(4, args.warmup + args.steps))]
    for s in range(args.warmup):
        idx, offs, go = batches[s % len(batches)]
        oracle.train_step(tables_h, off, wl.D, wl.B, idx, offs, go, scales, bits, wl.lr)
    t0 = time.perf_counter()
    lookups = 0
    for s in range(args.steps):
        idx, offs, go = batches[s % len(batches)]
        oracle.train_step(tables_h, off, wl.D, wl.B, idx, offs, go, scales, bits, wl.lr)
        lookups += len(idx)
    dt = time.perf_counter() - t0 + args.steps * t_refresh / wl.period
    value = lookups / dt
    sample = (f"{args.steps} full steps of batch {wl.B} (fwd+bwd+int8 quant+update) plus one whole-table "
              f"refresh of {wl.table_bytes() / 1e9:.2f} GB charged at 1/{wl.period} per step")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": base_config(wl),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2410_20046_b200 as dq

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dq.load_library()
    capture_stream = None
    if args.train_priority != 0:                     # the whole run, graph capture included, on a stream of that priority
        torch.cuda.set_stream(torch.cuda.Stream(priority=args.train_priority))
        capture_stream = torch.cuda.Stream(priority=args.train_priority)
    where = (rank, world, local_rank, capture_stream)

    line = measure(args, get_workload(args.workload), where, primary=True)
    # the other target configuration, measured in the same process (single GPU, default workload only)
    if world == 1 and args.workload == "kaggle_b16384" and not args.no_also:
        import copy
        a2 = copy.copy(args)
        a2.steps = min(args.steps, 500)
        import gc
        gc.collect()
        torch.cuda.empty_cache()                     # the first workload's tables and batches
        other = measure(a2, get_workload("terabyte_b32768"), where, primary=False)
        keys = ("value", "unit", "steps", "warmup", "ms_per_step", "config", "e2e", "gpu_launches", "roofline",
                "step_roofline", "kernel_rooflines", "kernels", "refresh")
        line["also"] = [{k: other[k] for k in keys}]
        if args.refresh_mode == "scan":
            # and the same configuration with the refresh fed from row summaries (an addition to the paper's
            # method that returns the same scales; the headline numbers above keep the refresh that scans)
            del other
            gc.collect()
            torch.cuda.empty_cache()
            a3 = copy.copy(a2)
            a3.refresh_mode = "summary"
            a3.e2e_steps = 0
            third = measure(a3, get_workload("terabyte_b32768"), where, primary=False)
            entry = {k: third[k] for k in keys if k != "e2e"}
            entry["variant"] = "refresh from per-row (min, max) summaries (--refresh-mode summary)"
            line["also"].append(entry)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def measure(args, wl, where, primary):
    """Times `args.steps` steps of workload `wl` on this rank's GPU and returns the JSON line as a dict."""
    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2410_20046_b200 as dq
    from dqrm_inputs import workloads as W
    from paper_2410_20046_b200 import harness

    rank, world, local_rank, capture_stream = where
    G = wl.T * wl.B
    tables = W.tables_torch(wl, "cuda")
    tables_h = tables.cpu().numpy() if (primary and rank == 0 and world == 1 and not args.no_cpu_baseline) else None

    # every rank is a full replica that takes its own B samples (weak scaling, no exchange)
    samplers = W.make_samplers(wl)
    batches = []
    for b in range(N_BATCHES):
        step_id = harness.batch_id(b, rank, world, N_BATCHES)
        idx, offs = W.make_batch(wl, step_id, samplers)
        offs_h = offs
        U = sum(len(np.unique(idx[offs_h[t * wl.B]:offs_h[(t + 1) * wl.B]])) for t in range(wl.T))
        batches.append(dict(L=len(idx), U=U, idx_h=torch.from_numpy(idx).pin_memory(),
                            off_h=torch.from_numpy(offs).pin_memory(),
                            go=W.grad_out_torch(wl, step_id, "cuda")))
    for b in batches:
        b["idx"], b["off"] = b["idx_h"].cuda(), b["off_h"].cuda()
        b["go_h"] = b["go"].cpu().pin_memory()
    Lmax = max(b["L"] for b in batches)
    Lavg = sum(b["L"] for b in batches) / N_BATCHES
    Uavg = sum(b["U"] for b in batches) / N_BATCHES

    ctx = dq.Context(wl.row_off(), wl.D, Lmax, G, host_step=True)
    ctx.set_overlap(not args.no_overlap)
    ctx.set_sort_path(args.sort_path)
    bits = torch.full((wl.T,), wl.bits, dtype=torch.int32, device="cuda")
    scales = torch.empty(wl.T, dtype=torch.float32, device="cuda")
    out = torch.empty((wl.B, wl.T, wl.D), dtype=torch.float32, device="cuda")
    out_h = torch.empty((wl.B, wl.T, wl.D), dtype=torch.float32).pin_memory()
    ur = torch.empty(Lmax, dtype=torch.int32, device="cuda")
    uo = torch.empty(wl.T + 1, dtype=torch.int32, device="cuda")
    gr = torch.empty((Lmax, wl.D), dtype=torch.float32, device="cuda")
    codes = torch.empty((Lmax, wl.D), dtype=torch.int8, device="cuda")
    gs = torch.empty(wl.T, dtype=torch.float32, device="cuda")

    summaries = args.refresh_mode == "summary"
    if summaries:       # per-row (min, max) kept current by the update kernels: a refresh reads 8 bytes per row
        ctx.row_summary_attach(tables)
    ctx.scale_refresh(tables, bits, scales)          # the steps before the first timed refresh use real scales too

    def launch_step(bi):
        b = batches[bi]
        ctx.train_step(tables, b["idx"], b["off"], b["go"], scales, bits, out, ur, uo, gr, codes, gs, wl.lr,
                       B=wl.B, L=b["L"])

    # Software pipeline over steps (default): the index half of the backward of batch k+1 (sort, unique rows)
    # runs on a second stream while batch k trains; the two halves hand over through two workspaces and two
    # (unique_rows, uniq_off) buffers used alternately.  Every step still does all of its own work inside the
    # timed region: K timed steps hold K sorts and K training halves.
    pipelined = not args.no_pipeline and not (args.dp_exchange and world > 1)
    if pipelined:
        assert N_BATCHES % 2 == 0
        side = torch.cuda.Stream(priority=args.sort_priority)
        ctx._workspace(1)                                   # allocate the second workspace before any capture
        urs = [ur, torch.empty_like(ur)]
        uos = [uo, torch.empty_like(uo)]

        def prime(bi):                                      # sorts batch bi ahead of its step (pipeline start)
            b = batches[bi]
            ctx.sort_batch(b["idx"], b["off"], urs[bi & 1], uos[bi & 1], B=wl.B, L=b["L"], ws=bi & 1)

        def launch_step(bi, join=True):     # noqa: F811
            b, nb, slot = batches[bi], batches[(bi + 1) % N_BATCHES], bi & 1
            cur = torch.cuda.current_stream()
            side.wait_stream(cur)
            if args.sort_after_forward:               # the sort runs beside the gradient summation and the update
                ctx.train_step_sorted(tables, b["idx"], b["off"], b["go"], scales, bits, out, urs[slot], uos[slot], gr,
                                      codes, gs, wl.lr, B=wl.B, L=b["L"], ws=slot, stream=cur)
                ctx.stream_wait_forward(side)
                ctx.sort_batch(nb["idx"], nb["off"], urs[slot ^ 1], uos[slot ^ 1], B=wl.B, L=nb["L"], ws=slot ^ 1,
                               stream=side)
            else:                                     # the sort runs beside the whole training half
                ctx.sort_batch(nb["idx"], nb["off"], urs[slot ^ 1], uos[slot ^ 1], B=wl.B, L=nb["L"], ws=slot ^ 1,
                               stream=side)
                ctx.train_step_sorted(tables, b["idx"], b["off"], b["go"], scales, bits, out, urs[slot], uos[slot], gr,
                                      codes, gs, wl.lr, B=wl.B, L=b["L"], ws=slot, stream=cur)
            # The next step's gradient summation waits for this sort by itself (an event the context keeps with the
            # workspace); its forward does not need the sort and may start before the sort is done.  Only the last
            # step of a captured graph joins the sort's stream (a capture must end with every stream joined).
            if join or args.join_every_step:
                cur.wait_stream(side)

        def launch_unpipelined(bi):
            b = batches[bi]
            ctx.train_step(tables, b["idx"], b["off"], b["go"], scales, bits, out, ur, uo, gr, codes, gs, wl.lr,
                           B=wl.B, L=b["L"])

    # The step is a fixed sequence of launches on fixed buffers, so each pre-staged batch's step is
    # captured once into a CUDA graph and replayed (the launches themselves are unchanged).
    dp_step = None
    if args.dp_exchange and world > 1:
        from paper_2410_20046_b200 import dp
        dp_step = dp.DataParallelStep(ctx, wl.B, Lmax, world)

        def launch_step(bi):     # noqa: F811  (the exchange has host-side size reads, so no graph capture)
            b = batches[bi]
            dp_step.step(tables, b["idx"], b["off"], b["go"], scales, bits, wl.lr, b["L"])
    graphs = None            # one CUDA graph per pre-staged batch: that batch's step
    group_graphs = None      # one CUDA graph per `spg` consecutive batches: their steps back to back
    launches_per_step = 0
    # steps per graph: whole groups must tile the batch ring and the refresh period; a timed region that is not a
    # whole number of groups ends with single-step graphs
    spg = args.steps_per_graph
    if spg < 1 or N_BATCHES % spg or wl.period % spg:
        spg = 1
    # shorter groups for the head and the tail of a timed region that the long groups do not tile
    group_sizes = [g for g in sorted({spg, 4}, reverse=True) if g > 1 and g <= spg and N_BATCHES % g == 0
                   and wl.period % g == 0]
    if not args.no_graph and dp_step is None:
        try:
            if pipelined:
                prime(0)
            for bi in range(2):
                launch_step(bi)                      # first use outside capture (function attributes, caches)
            torch.cuda.synchronize()

            def capture(first, count):
                if pipelined:
                    prime(first)                     # the graph's first step takes a sort made before the graph
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=capture_stream):
                    for bi in range(first, first + count):
                        if pipelined:
                            launch_step(bi, join=(bi == first + count - 1))
                        else:
                            launch_step(bi)
                return g

            n_before = ctx.launch_count()
            graphs = [capture(bi, 1) for bi in range(N_BATCHES)]
            launches_per_step = (ctx.launch_count() - n_before) // N_BATCHES    # kernels recorded per step
            if group_sizes:
                group_graphs = {g: [capture(b0, g) for b0 in range(0, N_BATCHES, g)] for g in group_sizes}
            torch.cuda.synchronize()
        except Exception as e:                       # capture refused: plain launches
            print(f"bench: CUDA graph capture failed ({e}); launching directly", file=sys.stderr)
            graphs = group_graphs = None
            torch.cuda.synchronize()

    last = {"s": None}
    refreshes = {"n": 0}     # scale refreshes launched since the timed region began

    def step(s, end=None, direct=False):
        """Runs step s, or a group of consecutive steps from one graph when they all lie before `end`; returns how many."""
        if s % wl.period == 0:
            ctx.scale_refresh(tables, bits, scales)
            refreshes["n"] += 1
        if direct and pipelined:                     # the per-kernel timing pass: one stream, one call per step
            launch_unpipelined(s % N_BATCHES)
            last["s"] = None
            return 1
        if pipelined and last["s"] != s - 1:
            prime(s % N_BATCHES)                     # (re)start of the pipeline: this batch is not sorted yet
        if group_graphs is not None and not direct and end is not None:
            for g in group_sizes:                    # the longest group that starts here and ends before `end`
                if s % g == 0 and s + g <= end:
                    group_graphs[g][(s % N_BATCHES) // g].replay()     # no refresh falls inside: g divides the period
                    last["s"] = s + g - 1
                    return g
        last["s"] = s
        if graphs is not None and not direct:
            graphs[s % N_BATCHES].replay()
        else:
            launch_step(s % N_BATCHES)
        return 1

    def step_host(s, end=None):
        if s % wl.period == 0:
            ctx.scale_refresh(tables, bits, scales)
        b = batches[s % N_BATCHES]
        ctx.train_step_host(tables, b["idx_h"], b["off_h"], b["go_h"], scales, bits, out_h, wl.lr, B=wl.B, L=b["L"])
        return 1

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def timed(fn, steps, warmup, sample_clocks=False):
        s = 0
        while s < warmup:
            s += fn(s, warmup)
        sync_all()
        sampler = ClockSampler(local_rank) if (sample_clocks and rank == 0) else None
        if sampler:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = ctx.launch_count()
        refreshes["n"] = 0
        e0.record()
        while s < warmup + steps:                      # exactly `steps` steps: s never passes the end
            s += fn(s, warmup + steps)
        e1.record()
        sync_all()
        ms = e0.elapsed_time(e1)
        clocks = sampler.stop() if sampler else None
        launches = ctx.launch_count() - n0             # direct launches (refresh; the steps too without graphs)
        if graphs is not None and fn is step:
            launches += steps * launches_per_step      # kernels replayed from the graphs
        ms = harness.max_over_ranks(ms, device="cuda")
        return ms, clocks, launches

    warm = max(3, args.warmup)
    ms, clocks, launches = timed(step, args.steps, warm, sample_clocks=primary)
    timed_refreshes = refreshes["n"]
    ctx.raise_on_device_error()
    lookups_per_step = Lavg * world
    value = harness.job_throughput(Lavg, world, args.steps, ms)

    e2e_steps = max(3, min(args.steps, args.e2e_steps))
    ms_e2e, _, _ = timed(step_host, e2e_steps, 3)
    ctx.raise_on_device_error()
    e2e_value = lookups_per_step * e2e_steps / (ms_e2e * 1e-3)
    h2d = int(4 * Lavg + 4 * (G + 1) + 4 * G * wl.D)
    d2h = int(4 * G * wl.D)

    # per-kernel times: a second pass over the same steps with an event after every launch
    prof_steps = min(args.steps, 200)
    for s in range(3):
        step(s)
    torch.cuda.synchronize()
    ctx.profile_begin()
    ctx.scale_refresh(tables, bits, scales)          # one refresh is always among the profiled launches
    for s in range(prof_steps):
        step(warm + s, direct=True)
    prof = ctx.profile_end()
    total_prof_ms = sum(v[0] for v in prof.values())
    kernels = {k: {"launches": v[1], "ms_total": round(v[0], 4), "us_per_launch": round(1e3 * v[0] / v[1], 3),
                   "share": round(v[0] / total_prof_ms, 4)} for k, v in sorted(prof.items(), key=lambda kv: -kv[1][0])}

    peak, peak_kind = measured_peak()
    ab = algorithmic_bytes(wl, Lavg, G, Uavg)
    if summaries:       # what that refresh reads, and what the updates write on top of the rows
        ab["refresh"] = 8 * int(wl.row_off()[-1])
        ab["quant_update"] += 8 * Uavg
        ab["step"] += 8 * Uavg
        ab["step_separate_calls"] += 8 * Uavg
    dominant = max((k for k in prof if k in KERNEL_BYTES), key=lambda k: prof[k][0])
    dom_bytes = KERNEL_BYTES[dominant](ab, wl, Lavg, G, Uavg)
    dom_s = prof[dominant][0] * 1e-3 / prof[dominant][1]
    achieved = dom_bytes / dom_s / 1e9
    per_kernel_roofline = {}
    for k in prof:
        if k in KERNEL_BYTES:
            by = KERNEL_BYTES[k](ab, wl, Lavg, G, Uavg)
            gbs = by / (prof[k][0] * 1e-3 / prof[k][1]) / 1e9
            per_kernel_roofline[k] = {"algorithmic_bytes": int(by), "GB/s": round(gbs, 1),
                                      "frac_of_" + peak_kind: round(gbs / peak, 4)}
    # bytes of the timed region: the steps, plus the whole-table reads of the refreshes that ran inside it
    step_bytes = ab["step"] + ab["refresh"] * timed_refreshes / args.steps
    step_bytes_sep = ab["step_separate_calls"] + ab["refresh"] * timed_refreshes / args.steps
    s_per_step = ms * 1e-3 / args.steps
    step_gbs = step_bytes / s_per_step / 1e9                      # per GPU: every rank moves these bytes in that time
    step_gbs_sep = step_bytes_sep / s_per_step / 1e9
    # the refresh by itself, and the step time with one refresh charged every `period` steps whatever --steps was
    refresh_us = 1e3 * prof["refresh_kernel"][0] / prof["refresh_kernel"][1] if "refresh_kernel" in prof else None
    steps_only_us = (ms * 1e3 - (refresh_us or 0.0) * timed_refreshes) / args.steps
    amortised_us = steps_only_us + (refresh_us or 0.0) / wl.period
    amortised_bytes = ab["step"] + ab["refresh"] / wl.period

    cpu_baseline = None
    if tables_h is not None:
        n = args.cpu_steps if args.cpu_steps > 0 else cpu_sample_steps(wl)
        (v, t_step, t_ref), (v_mc, t_step_mc, t_ref_mc, threads, cores) = oracle_sample(wl, tables_h, n, wl.period)
        sample = (f"{n} full steps of batch {wl.B} ({{:.0f}} ms each) plus one whole-table refresh ({{:.0f}} ms) "
                  f"charged at 1/{wl.period} per step")
        cpu_baseline = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
                        "sample": sample.format(t_step * 1e3, t_ref * 1e3),
                        "all_cores": {"value": v_mc, "unit": UNIT, "cores": threads, "host_cores": cores,
                                      "kind": "oracle, one table per thread",
                                      "sample": sample.format(t_step_mc * 1e3, t_ref_mc * 1e3)}}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warm, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": base_config(wl),
        "run": {"lookups_per_step_per_gpu": Lavg, "unique_rows_per_step": Uavg, "unique_fraction": Uavg / Lavg,
                "launch": ((f"CUDA graph replay, groups of {group_sizes} consecutive steps per graph, single steps "
                            "for the rest" if group_graphs is not None else "CUDA graph replay per step")
                           if graphs is not None else "direct launches") +
                          ("; the index sort of batch k+1 runs on a second stream while batch k trains "
                           "(two workspaces, every step does one sort and one training half)" if pipelined
                           else ""),
                "parallelism": (f"{world} ranks, sparse INT8 gradient exchange every step" if dp_step is not None
                                else f"{world} replica(s), batch sharded by sample, no exchange"),
                "l2": f"{N_BATCHES} distinct pre-staged batches cycled; their rows, gradients and outputs "
                      f"exceed the 126 MB L2 and the table is {wl.table_bytes() / 1e9:.2f} GB",
                "refreshes_in_timed_region": timed_refreshes},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": dominant, "achieved": round(achieved, 1), "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": round(achieved / peak, 4),
                     "frac_of_8TBps_nominal": round(achieved / NOMINAL_HBM_GBS, 4),
                     "traffic": NCU_TRAFFIC.get((wl.name, dominant)),
                     "algorithmic_bytes_per_launch": int(dom_bytes)},
        # the timed region as it ran: its steps and the refreshes that fell inside it, bytes over time
        "step_roofline": {"algorithmic_bytes_per_step": int(step_bytes), "GB/s": round(step_gbs, 1),
                          "frac_of_" + peak_kind: round(step_gbs / peak, 4),
                          "frac_of_8TBps_nominal": round(step_gbs / NOMINAL_HBM_GBS, 4),
                          "separate_calls_bytes_per_step": int(step_bytes_sep),
                          "separate_calls_frac_of_" + peak_kind: round(step_gbs_sep / peak, 4),
                          "separate_calls_frac_of_8TBps_nominal": round(step_gbs_sep / NOMINAL_HBM_GBS, 4)},
        # the same with one refresh charged every `period` steps (its own measured time and its bytes), whatever
        # --steps was
        "refresh": {"mode": ("per-row (min, max) summaries, 8 bytes per row, kept current by the update kernels"
                             if summaries else "scan of the tables"),
                    "us": None if refresh_us is None else round(refresh_us, 2), "bytes": int(ab["refresh"]),
                    "period": wl.period, "us_per_step_amortised": round(amortised_us, 3),
                    "lookups_per_s_amortised": Lavg * world / (amortised_us * 1e-6),
                    "bytes_per_step_amortised": int(amortised_bytes),
                    "frac_of_" + peak_kind: round(amortised_bytes / (amortised_us * 1e-6) / 1e9 / peak, 4),
                    "frac_of_8TBps_nominal": round(amortised_bytes / (amortised_us * 1e-6) / 1e9 / NOMINAL_HBM_GBS, 4)},
        "kernel_rooflines": per_kernel_roofline,
        "kernels": kernels,
        "cpu_baseline": cpu_baseline,
    }
    ctx.close()
    torch.cuda.synchronize()
    return line


def run_packed(args):
    """Appendix C, the deployed form: bit-pack the quantised tables once, then serve lookups from the
    packed arena.  One JSON line: lookups/s of the packed forward, and the two kernels against the
    HBM roofline on their algorithmic bytes."""
    import numpy as np
    import torch

    import paper_2410_20046_b200 as dq
    from dqrm_inputs import workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    wl = get_workload(args.workload)
    G = wl.T * wl.B
    bits_w = wl.bits if wl.bits in (2, 4, 8) else 4
    tables = W.tables_torch(wl, "cuda")
    samplers = W.make_samplers(wl)
    batches = []
    for b in range(N_BATCHES):
        idx, offs = W.make_batch(wl, b, samplers)
        U = sum(len(np.unique(idx[offs[t * wl.B]:offs[(t + 1) * wl.B]])) for t in range(wl.T))
        batches.append(dict(L=len(idx), U=U, idx=torch.from_numpy(idx).cuda(), off=torch.from_numpy(offs).cuda()))
    Lavg = sum(b["L"] for b in batches) / N_BATCHES
    Uavg = sum(b["U"] for b in batches) / N_BATCHES
    ctx = dq.Context(wl.row_off(), wl.D, max(b["L"] for b in batches), G)
    bits = torch.full((wl.T,), bits_w, dtype=torch.int32, device="cuda")
    scales = torch.empty(wl.T, dtype=torch.float32, device="cuda")
    ctx.scale_refresh(tables, bits, scales)
    packed = torch.empty(ctx.packed_bytes(bits_w), dtype=torch.uint8, device="cuda")
    out = torch.empty((wl.B, wl.T, wl.D), dtype=torch.float32, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    for _ in range(3):
        ctx.pack_tables(tables, scales, bits_w, packed)
    n_pack = 10
    e0.record()
    for _ in range(n_pack):
        ctx.pack_tables(tables, scales, bits_w, packed)
    e1.record()
    torch.cuda.synchronize()
    pack_ms = e0.elapsed_time(e1) / n_pack
    pack_bytes = tables.numel() * 4 + packed.numel()

    def lookup(b):
        ctx.packed_fwd(packed, b["idx"], b["off"], scales, bits_w, out, B=wl.B, L=b["L"])

    for b in batches[:3]:
        lookup(b)
    torch.cuda.synchronize()
    graphs = []
    for b in batches:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            lookup(b)
        graphs.append(g)
    warm = max(3, args.warmup)
    for s in range(warm):
        graphs[s % N_BATCHES].replay()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    e0.record()
    for s in range(args.steps):
        graphs[(warm + s) % N_BATCHES].replay()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    ctx.raise_on_device_error()
    peak, peak_kind = measured_peak()
    fwd_bytes = 4 * Lavg + 4 * G + Uavg * wl.D * bits_w / 8 + 4 * wl.D * G
    fwd_gbs = fwd_bytes / (ms * 1e-3 / args.steps) / 1e9
    pack_gbs = pack_bytes / (pack_ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "packed embedding lookups/sec (inference from the bit-packed tables)",
        "value": Lavg * args.steps / (ms * 1e-3), "unit": "lookups/s", "n_gpus": 1, "steps": args.steps, "warmup": warm,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": f"int{bits_w} codes, f32 output", "data": "synthetic",
        "config": {"workload": wl.name, "tables": wl.T, "dim": wl.D, "batch_per_gpu": wl.B, "bits": bits_w,
                   "packed_bytes": int(packed.numel()), "table_bytes": wl.table_bytes(),
                   "launch": "CUDA graph replay per batch", "l2": f"{N_BATCHES} distinct batches cycled"},
        "gpu_launches": int(args.steps), "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": "packed_fwd_kernel", "achieved": round(fwd_gbs, 1), "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": round(fwd_gbs / peak, 4), "traffic": None,
                     "algorithmic_bytes_per_launch": int(fwd_bytes)},
        "pack_kernel": {"ms": round(pack_ms, 4), "algorithmic_bytes": int(pack_bytes), "GB/s": round(pack_gbs, 1),
                        "frac_of_" + peak_kind: round(pack_gbs / peak, 4)},
    }))
    ctx.close()


def launch_ranks(args):
    """--gpus N without a launcher in the environment: start N ranks of this script, one per GPU, the way
    the contract's launcher does, and pass their output through.  NCCL's initialisation log goes to files
    of a temporary folder; its communicator lines are echoed to stderr afterwards."""
    import glob
    import socket
    import tempfile

    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = dict(os.environ)
    logdir = tempfile.mkdtemp(prefix="dqrm_nccl_")
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    env.setdefault("NCCL_DEBUG_FILE", os.path.join(logdir, "nccl.%h.%p.log"))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    rc = subprocess.call(cmd, env=env, cwd=ROOT)
    shown = 0
    for f in sorted(glob.glob(os.path.join(logdir, "*.log"))):
        with open(f, errors="replace") as fh:
            for ln in fh:
                if shown < 60 and any(k in ln for k in ("Init COMPLETE", "NVLS", "comm 0x", "Connected all")):
                    print("nccl:", ln.rstrip(), file=sys.stderr)
                    shown += 1
    return rc


def run_stub(args):
    """Launcher and rendezvous check without a GPU (used by the CPU tests): every rank sleeps through its
    steps on the gloo backend, the job's time is the slowest rank's, rank 0 prints the line."""
    import torch.distributed as dist
    from paper_2410_20046_b200 import harness

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.002 * (1 + rank))
    ms = harness.max_over_ranks((time.perf_counter() - t0) * 1e3)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": harness.job_throughput(1000, world, args.steps, ms), "unit": UNIT,
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
                          "higher_is_better": True, "scaling": "weak", "stub": True}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-pipeline", action="store_true",
                    help="one dqrm_train_step call per step instead of sorting the next batch beside the current one")
    ap.add_argument("--packed", action="store_true",
                    help="time the bit-packed export and the packed inference lookup instead of the training step")
    ap.add_argument("--workload", default="kaggle_b16384")
    ap.add_argument("--e2e-steps", type=int, default=50)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true",
                    help="with the default workload: do not measure terabyte_b32768 as well")
    ap.add_argument("--dp-exchange", action="store_true",
                    help="with --gpus N > 1: exchange the sparse INT8 gradient every step (paper's data parallelism) "
                         "instead of running independent replicas")
    ap.add_argument("--no-graph", action="store_true", help="launch every step directly instead of replaying CUDA graphs")
    ap.add_argument("--no-overlap", action="store_true", help="keep the index sort on the caller's stream")
    ap.add_argument("--steps-per-graph", type=int, default=20,
                    help="consecutive steps replayed from one CUDA graph (must divide the 20 staged batches and the refresh period, else 1; "
                         "a remainder of the timed region runs from single-step graphs)")
    ap.add_argument("--sort-priority", type=int, default=0,
                    help="priority of the second stream that sorts the next batch (-1 high, 0 default)")
    ap.add_argument("--train-priority", type=int, default=-1,
                    help="priority of the stream the training half runs on (0: torch's current stream)")
    ap.add_argument("--sort-after-forward", type=int, default=0,
                    help="1: the next batch's sort waits for this batch's forward and runs beside the rest of the step")
    ap.add_argument("--cpu-steps", type=int, default=0,
                    help="full steps the CPU oracle is timed on (0: as many as make about ten seconds on one core)")
    ap.add_argument("--refresh-mode", choices=("scan", "summary"), default="scan",
                    help="scan: every refresh reads the whole tables (the paper's refresh); summary: the library keeps "
                         "(min, max) of every row current as it updates rows and a refresh reads those, same scales")
    ap.add_argument("--join-every-step", action="store_true",
                    help="make every step wait for the next batch's sort before the following step begins "
                         "(default: only that step's gradient summation waits; its forward starts at once)")
    ap.add_argument("--sort-path", type=int, default=0, help="0: per-table cluster sort, 1: global radix sort")
    ap.add_argument("--stub-step", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours" and not args.packed:
        sys.exit(launch_ranks(args))
    if args.stub_step:
        run_stub(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.packed:
        run_packed(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
