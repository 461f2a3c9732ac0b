"""bench.py's launch path on a CPU-only box: `--gpus N` without a launcher starts N ranks itself
(torch.distributed.run on 127.0.0.1; gloo when there is no GPU) and the line says how many ranks ran."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args, env_extra=None, timeout=300):
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env.update(env_extra or {})
    env["CUDA_VISIBLE_DEVICES"] = ""                      # the launch path is what is under test, not the GPU
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                       timeout=timeout, env=env, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [json.loads(l) for l in p.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, p.stdout                       # rank 0 alone prints
    return lines[0]


def test_gpus_flag_starts_that_many_ranks():
    line = _run("--gpus", "2", "--dry-run")
    assert line["n_gpus"] == 2 and line["ranks"] == [0, 1] and line["scaling"] == "weak"
    assert "dp2" in line["config"]["parallelism"]


def test_single_rank_dry_run():
    line = _run("--dry-run")
    assert line["n_gpus"] == 1 and line["ranks"] == [0]


def test_world_size_mismatch_fails_loudly():
    env = {k: v for k, v in os.environ.items()}
    env.update(WORLD_SIZE="1", RANK="0", LOCAL_RANK="0", CUDA_VISIBLE_DEVICES="")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--dry-run"], capture_output=True,
                       text=True, timeout=120, env=env, cwd=ROOT)
    assert p.returncode != 0 and "--gpus 4" in p.stderr
