"""bench.py's command line without a GPU: the reference arm (the oracle on host cores) prints the contract's
JSON line, and `--gpus N` outside a torchrun environment starts N ranks itself, of which rank 0 alone works."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*flags):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1",
                        "--steps", "2", "--warmup", "1", "--ref-rows", "8", *flags],
                       capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout[-2000:]            # one JSON line, from rank 0 only
    return json.loads(lines[0])


def _check(line, n):
    assert line["impl"] == "reference" and line["n_gpus"] == n and line["steps"] == 2
    assert line["value"] > 0 and line["unit"] == "positions/s" and line["higher_is_better"] is True
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"]["value"] == line["value"] and line["e2e"]["h2d_bytes_per_step"] == 0
    assert "workload" in line["config"] and "model" not in line["config"]


def test_reference_arm_prints_the_contract_line():
    _check(_run(), 1)


def test_gpus_flag_starts_the_ranks_itself():
    _check(_run("--gpus", "2"), 2)
