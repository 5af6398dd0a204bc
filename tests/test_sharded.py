"""Group-sharded rollout: the partition of groups over ranks and the final gather, on CPU
(gloo, world size 2 and 3).  The per-rank results are a deterministic function of the *global*
group id, standing in for the GPU rollout, whose random streams are keyed the same way."""
import os
import socket
import subprocess
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(HERE))
from paper_2601_19404_b200 import sharded


def test_partition_is_exact_balanced_and_deterministic():
    rng = np.random.default_rng(0)
    lens = rng.integers(1024, 6145, size=64)
    for world in (1, 2, 3, 8):
        parts = sharded.partition_groups(lens, 8, 256, world)
        assert len(parts) == world
        allg = np.concatenate(parts)
        assert np.array_equal(np.sort(allg), np.arange(64))              # every group exactly once
        assert all(np.all(np.diff(p) > 0) for p in parts if p.size > 1)  # ascending within a rank
        cost = lens + 8 * 256
        loads = np.array([cost[p].sum() for p in parts])
        assert loads.max() - loads.min() <= cost.max()                   # longest-first greedy bound
        again = sharded.partition_groups(lens, 8, 256, world)
        assert all(np.array_equal(a, b) for a, b in zip(parts, again))
    assert np.array_equal(sharded.partition_groups(lens, 8, 256, 1)[0], np.arange(64))
    few = sharded.partition_groups([10, 20], 4, 8, 3)                    # more ranks than groups
    assert sorted(len(p) for p in few) == [0, 1, 1]


def test_gather_without_process_group_is_identity():
    G, S, n = 2, 3, 4
    tok = np.arange(n * G * S, dtype=np.int32).reshape(n * G, S)
    out = sharded.gather_rollout({"tokens": tok, "lens": np.full(n * G, S, np.int32), "logprobs": None}, np.arange(n), n, G, S)
    assert np.array_equal(out["tokens"], tok) and "logprobs" not in out


WORKER = r"""
import os, sys
import numpy as np
import torch, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
from paper_2601_19404_b200 import sharded
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, world = dist.get_rank(), dist.get_world_size()
G, S, n_g = 4, 6, 7
lens = np.array([900, 100, 500, 2000, 50, 700, 300])

def fake(g):      # result of group g: depends on the global id only
    i = np.arange(G)[:, None]; j = np.arange(S)[None, :]
    tok = (g * 1000 + i * 10 + j).astype(np.int32)
    ln = ((g + np.arange(G)) % S + 1).astype(np.int32)
    lp = -(tok.astype(np.float32)) / 7.0
    return tok, ln, lp

owned = sharded.partition_groups(lens, G, S, world)[rank]
parts = [fake(int(g)) for g in owned]
local = {"tokens": np.concatenate([p[0] for p in parts]) if parts else np.zeros((0, S), np.int32),
         "lens": np.concatenate([p[1] for p in parts]) if parts else np.zeros(0, np.int32),
         "logprobs": np.concatenate([p[2] for p in parts]) if parts else np.zeros((0, S), np.float32)}
out = sharded.gather_rollout(local, owned, n_g, G, S)
for g in range(n_g):
    tok, ln, lp = fake(g)
    assert np.array_equal(out["tokens"][g * G:(g + 1) * G], tok)
    assert np.array_equal(out["lens"][g * G:(g + 1) * G], ln)
    assert np.array_equal(out["logprobs"][g * G:(g + 1) * G], lp)
# a group claimed twice is an error on every rank
try:
    sharded.gather_rollout({"tokens": np.zeros((G, S), np.int32), "lens": np.zeros(G, np.int32), "logprobs": None}, [0], n_g, G, S)
    raise SystemExit("duplicate ownership not detected")
except ValueError:
    pass
print("OK", rank)
dist.destroy_process_group()
"""


def _run(world, tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), os.path.dirname(HERE)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=240)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert all("OK" in o for o in outs)


def test_gather_over_two_gloo_ranks(tmp_path):
    _run(2, tmp_path)


def test_gather_over_three_gloo_ranks(tmp_path):
    _run(3, tmp_path)
