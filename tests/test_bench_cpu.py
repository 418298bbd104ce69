"""The reference arm of bench.py (the oracle timed on the host cores) needs no GPU: its JSON line
must carry the contract's keys, and the product arm must refuse to run without a CUDA device."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args, env=None):
    e = dict(os.environ)
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                          cwd=ROOT, env=e, timeout=600)


def test_reference_arm_prints_the_contract_line():
    r = _run("--impl", "reference", "--workload", "tiny", "--steps", "3", "--warmup", "1")
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["unit"] == "lookups/s" and j["higher_is_better"] is True
    assert j["steps"] == 3 and j["warmup"] == 1 and j["value"] > 0 and j["vs_baseline"] is None
    assert j["config"]["workload"] == "tiny"
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["value"] == j["value"]
    assert j["e2e"] == {"value": j["value"], "unit": j["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_reference_arm_other_ranks_do_nothing():
    r = _run("--impl", "reference", "--workload", "tiny", "--steps", "1", "--warmup", "0", env={"RANK": "1"})
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_product_arm_fails_loudly_without_a_gpu():
    import torch

    if torch.cuda.is_available():
        return
    r = _run("--workload", "tiny", "--steps", "1")
    assert r.returncode != 0
    assert "CUDA" in (r.stderr + r.stdout)


def test_gpus_flag_starts_that_many_ranks_itself():
    """`--gpus 2` with no launcher in the environment: the script starts two ranks (gloo stand-in step on CPU),
    rank 0 prints the one line, and the job's time is the slower rank's."""
    env = {k: "" for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    e = {k: v for k, v in os.environ.items() if k not in env}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "5", "--warmup", "0",
                        "--stub-step"], capture_output=True, text=True, cwd=ROOT, env=e, timeout=600)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout
    j = json.loads(lines[0])
    assert j["n_gpus"] == 2 and j["steps"] == 5
    assert j["ms_per_step"] >= 4.0            # rank 1 sleeps 4 ms per step, rank 0 only 2
    assert abs(j["value"] - 1000 * 2 / (j["ms_per_step"] * 1e-3)) < 1e-6 * j["value"]


def test_all_cores_oracle_sample_is_the_same_computation():
    """The benchmark's all-cores CPU figure runs the oracle on one-table problems, a thread each: it must leave
    the tables exactly as the single call does."""
    import numpy as np
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    from dqrm_inputs import workloads as W

    oracle.build()
    wl = W.tiny()
    off = wl.row_off()
    bits = np.full(wl.T, wl.bits, dtype=np.int32)
    idx, offs = W.make_batch(wl, 0)
    go = W.grad_out_np(wl, 0)
    whole = W.tables_np(wl)
    scales, _ = oracle.scale_refresh(whole, off, wl.D, bits)
    split = whole.copy()
    oracle.train_step(whole, off, wl.D, wl.B, idx, offs, go, scales, bits, wl.lr)

    def one(t):
        lo, hi = offs[t * wl.B], offs[(t + 1) * wl.B]
        s1, _ = oracle.scale_refresh(split[off[t]:off[t + 1]], np.array([0, off[t + 1] - off[t]]), wl.D, bits[t:t + 1])
        assert s1[0] == scales[t]
        oracle.train_step(split[off[t]:off[t + 1]], np.array([0, off[t + 1] - off[t]], dtype=np.int64), wl.D, wl.B,
                          np.ascontiguousarray(idx[lo:hi]), np.ascontiguousarray(offs[t * wl.B:(t + 1) * wl.B + 1] - lo),
                          np.ascontiguousarray(go[:, t:t + 1, :]), scales[t:t + 1], bits[t:t + 1], wl.lr)

    with ThreadPoolExecutor(max_workers=4) as pool:
        list(pool.map(one, range(wl.T)))
    assert split.tobytes() == whole.tobytes()
