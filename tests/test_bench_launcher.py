"""`python bench.py --gpus N` without a launcher starts N ranks by itself.  Checked on the host:
the ranks meet over gloo (no GPU work) and rank 0 reports how many came."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_selfcheck(n):
    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", str(n),
                          "--selfcheck-ranks"], capture_output=True, text=True, env=env,
                         timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    return json.loads(lines[0])


def test_bench_starts_its_own_ranks():
    rec = run_selfcheck(2)
    assert rec["n_gpus"] == 2 and rec["world_size"] == 2


def test_bench_single_rank_needs_no_launcher():
    rec = run_selfcheck(1)
    assert rec["n_gpus"] == 1 and rec["world_size"] == 1
