"""Host-side checks of the synthetic workloads: shape of config 5 against the token counts the
paper prints, determinism of the generators, and group sharding over ranks (gloo, world size 2)."""
import os
import socket
import subprocess
import sys

import numpy as np

import workloads

HERE = os.path.dirname(os.path.abspath(__file__))


def _golden():
    rows = {}
    for line in open(os.path.join(HERE, "golden", "avg_generated_tokens.txt")):
        if line.strip() and not line.startswith("#"):
            k, a, b = line.split()
            rows[k] = (float(a), float(b))
    return rows


def test_config5_generated_token_ratio_lies_in_the_papers_range():
    g = _golden()
    ratios = [g[k][m] / g["GRPO"][m] for k in ("L=300", "L=500", "L=800") for m in (0, 1)]
    part, full = workloads.CONFIGS["cfg5_7b_partial"], workloads.CONFIGS["cfg5_7b_full"]
    ratio = part["suffix"] / full["suffix"]
    assert min(ratios) <= ratio <= max(ratios)          # 5.4 % .. 16.2 % in the paper, 5.9 % here
    assert abs(full["suffix"] - np.mean([g["GRPO"][0], g["GRPO"][1]])) < 2000   # same order as the full-path mean


def test_generators_are_seeded_and_shaped():
    cfg = workloads.CONFIGS["cfg3_1p5b_64x8_ragged"]
    a, b = workloads.prefix_lengths(cfg, seed=0), workloads.prefix_lengths(cfg, seed=0)
    assert np.array_equal(a, b) and a.min() >= 1024 and a.max() <= 6144 and len(a) == 64
    assert not np.array_equal(a, workloads.prefix_lengths(cfg, seed=1))
    t, off = workloads.prefix_tokens(a, 151936, seed=0)
    assert off[-1] == a.sum() == len(t) and t.min() >= 0 and t.max() < 151936
    assert np.array_equal(workloads.rank_group_ids(4, rank=3), np.arange(12, 16))


WORKER = r"""
import os, sys
import numpy as np
import torch, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
import workloads
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, world = dist.get_rank(), dist.get_world_size()
cfg = workloads.CONFIGS["cfg3_1p5b_64x8_ragged"]
n_g = 6
ids = workloads.rank_group_ids(n_g, rank)
lens = workloads.prefix_lengths(cfg, seed=rank, n_groups=n_g)
# what bench.py reduces over ranks: MAX of the times, SUM of the emitted tokens
t = torch.tensor([10.0 + rank], dtype=torch.float64); dist.all_reduce(t, op=dist.ReduceOp.MAX)
em = torch.tensor([int(lens.sum())], dtype=torch.int64); dist.all_reduce(em, op=dist.ReduceOp.SUM)
gathered = [torch.zeros(n_g, dtype=torch.int64) for _ in range(world)]
dist.all_gather(gathered, torch.from_numpy(ids.astype(np.int64)))
if rank == 0:
    all_ids = torch.cat(gathered).numpy()
    assert len(set(all_ids.tolist())) == n_g * world, "group ids (hence random streams) must not overlap across ranks"
    expect = sum(int(workloads.prefix_lengths(cfg, seed=r, n_groups=n_g).sum()) for r in range(world))
    assert int(em.item()) == expect and t.item() == 10.0 + world - 1
    print("OK")
dist.destroy_process_group()
"""


def test_group_sharding_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), os.path.dirname(HERE)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=240)[0] for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    assert "OK" in outs[0]
