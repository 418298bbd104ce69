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
