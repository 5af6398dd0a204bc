"""Group-sharded rollout over several GPUs, one process per GPU (torch.distributed).

Prompt groups are independent: the G samples of a question depend only on that question's prefix
(Eq. 3; Algorithm 1's rollout loop), which is also how the paper spreads its cache initialisation
over GPUs (Section 4.1).  So the groups are partitioned over the ranks, every rank holds the same
weights (same seed -> identical initialisation, nothing is broadcast), prefill and decode run with no
collective at all, and one all_gather at the end gives every rank the whole batch.  A group keeps
its *global* id on whichever rank it lands, and the sampler's random stream is keyed by
(seed, group_id * G + i, step): the result does not depend on the number of ranks.
"""
import numpy as np


def partition_groups(prefix_lens, G, max_new, world):
    """Groups -> ranks, balanced by the cost model sum(P_g + G * max_new): longest-first greedy.
    Returns `world` ascending int64 index arrays that partition range(len(prefix_lens))."""
    prefix_lens = np.asarray(prefix_lens, dtype=np.int64)
    cost = prefix_lens + int(G) * int(max_new)
    order = np.argsort(-cost, kind="stable")
    load = np.zeros(world, dtype=np.int64)
    parts = [[] for _ in range(world)]
    for g in order:
        r = int(np.argmin(load))           # lowest rank among the least loaded
        parts[r].append(int(g)); load[r] += cost[g]
    return [np.asarray(sorted(p), dtype=np.int64) for p in parts]


def gather_rollout(local, owned, n_groups, G, max_new, group=None):
    """All-gather of the per-rank results into global group order.

    local: dict with 'tokens' [n_local*G, max_new] int32, 'lens' [n_local*G] int32 and optionally
    'logprobs' [n_local*G, max_new] float32 (numpy or torch, any device) for the groups `owned`
    (ascending global indices, this rank's part).  Every rank returns the same dict of numpy arrays
    for all n_groups groups."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    backend = dist.get_backend(group) if dist.is_initialized() else "none"
    dev = torch.device("cuda", torch.cuda.current_device()) if backend == "nccl" else torch.device("cpu")
    owned = np.asarray(owned, dtype=np.int64)
    n_local = owned.size
    cap = -(-n_groups // world) if world > 1 else n_groups          # a rank owns at most ceil(n/world) groups + slack
    if world > 1:
        t = torch.tensor([n_local], dtype=torch.int64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
        cap = int(t.item())

    def pad(x, dtype, cols):
        x = torch.as_tensor(x).to(dev).to(dtype).reshape(n_local * G, *cols)
        out = torch.zeros((cap * G, *cols), dtype=dtype, device=dev)
        out[:n_local * G] = x
        return out

    ids = torch.full((cap,), -1, dtype=torch.int64, device=dev)
    ids[:n_local] = torch.from_numpy(owned).to(dev)
    send = {"ids": ids, "tokens": pad(local["tokens"], torch.int32, (max_new,)), "lens": pad(local["lens"], torch.int32, ())}
    if local.get("logprobs") is not None:
        send["logprobs"] = pad(local["logprobs"], torch.float32, (max_new,))
    got = {}
    for k, v in send.items():
        if world > 1:
            bufs = [torch.zeros_like(v) for _ in range(world)]
            dist.all_gather(bufs, v, group=group)
        else:
            bufs = [v]
        got[k] = [b.cpu().numpy() for b in bufs]
    out = {"tokens": np.zeros((n_groups * G, max_new), dtype=np.int32), "lens": np.zeros(n_groups * G, dtype=np.int32)}
    if "logprobs" in got:
        out["logprobs"] = np.zeros((n_groups * G, max_new), dtype=np.float32)
    seen = np.zeros(n_groups, dtype=bool)
    for r in range(world):
        for j, g in enumerate(got["ids"][r]):
            if g < 0:
                continue
            if seen[g]:
                raise ValueError(f"group {g} is owned by more than one rank")
            seen[g] = True
            for k in out:
                out[k][g * G:(g + 1) * G] = got[k][r][j * G:(j + 1) * G]
    if not seen.all():
        raise ValueError("some groups are owned by no rank")
    return out


def sharded_rollout(ctx, sampler, prefixes, G, max_new, want_logprobs=True, group=None):
    """Rolls out G suffixes for every prefix in `prefixes` (list of int32 arrays, identical on all
    ranks) with the groups partitioned over the ranks of `group`; returns the gathered batch
    (see gather_rollout).  `ctx` is this rank's paper_2601_19404_b200.Context."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    lens = np.asarray([len(p) for p in prefixes], dtype=np.int64)
    owned = partition_groups(lens, G, max_new, world)[rank]
    dev = torch.device("cuda", torch.cuda.current_device())
    n_local = owned.size
    d_out = torch.zeros((max(n_local, 1) * G, max_new), dtype=torch.int32, device=dev)
    d_lens = torch.zeros(max(n_local, 1) * G, dtype=torch.int32, device=dev)
    d_lp = torch.zeros((max(n_local, 1) * G, max_new), dtype=torch.float32, device=dev) if want_logprobs else None
    if n_local:
        off = np.zeros(n_local + 1, dtype=np.int32)
        off[1:] = np.cumsum(lens[owned])
        toks = np.concatenate([np.asarray(prefixes[g], dtype=np.int32) for g in owned])
        groups = ctx.prefill_prefix(torch.from_numpy(toks).to(dev), off, owned.astype(np.int32))   # global ids -> random streams
        ctx.decode_suffix(groups, G, max_new, sampler, d_out, d_lens, d_lp)
        ctx.release_groups(groups)
        torch.cuda.synchronize()
    local = {"tokens": d_out[:n_local * G], "lens": d_lens[:n_local * G], "logprobs": d_lp[:n_local * G] if want_logprobs else None}
    return gather_rollout(local, owned, len(prefixes), G, max_new, group)
