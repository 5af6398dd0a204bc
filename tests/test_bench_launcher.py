"""`python bench.py --gpus N` starts its N ranks itself.  The rank plumbing - spawning one process per
device, the rendezvous on 127.0.0.1, MAX over ranks of the timings, SUM of the token counts, rank 0's
single JSON line - is exercised here on CPU with the gloo backend (no GPU work)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(n):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", str(n), "--plumbing-only"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout                       # one JSON line, from rank 0 only
    return json.loads(lines[0])


def test_gpus_flag_spawns_the_ranks_and_reduces_over_them():
    two = _run(2)
    assert two["n_gpus"] == 2 and two["plumbing_only"]
    assert two["ms_per_step"] == 101.0 and two["other_ms"] == 20.0        # MAX over ranks of (100 + rank, 10 (rank + 1))
    assert two["tokens"] == 1000 + 1001                                    # SUM over ranks
    assert abs(two["value"] - 2001 / 0.101) < 1e-6
    one = _run(1)
    assert one["n_gpus"] == 1 and one["ms_per_step"] == 100.0 and one["tokens"] == 1000
