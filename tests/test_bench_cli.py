"""bench.py's command line without a GPU: `--gpus N` given without a launcher starts its own N ranks, and
the reference arm (the float64 oracle on the host cores) prints exactly one JSON line from rank 0."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*flags):
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--r", "8", "--steps", "2", "--warmup", "1", "--oracle-frac", "1", *flags],
                         capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    return [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]


def test_reference_arm_prints_one_line_with_the_contract_keys():
    lines = _run()
    assert len(lines) == 1
    d = lines[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 1 and d["steps"] == 2 and d["unit"] == "layers/s"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"] > 0
    assert d["e2e"] == {"value": d["value"], "unit": "layers/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    # a step is one bounded sample; value = layers per step / time per step
    assert abs(d["value"] - 1e3 * d["config"]["layers_per_step"] / d["ms_per_step"]) <= 1e-9 * d["value"]


def test_gpus_2_without_a_launcher_starts_its_own_ranks_and_rank_0_alone_prints():
    lines = _run("--gpus", "2")
    assert len(lines) == 1 and lines[0]["n_gpus"] == 2 and lines[0]["impl"] == "reference"
