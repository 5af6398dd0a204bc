"""Helpers shared by the GPU parity tests: context construction and oracle twins."""
import numpy as np
import torch

import paper_2601_19404_b200 as rpo
from paper_2601_19404_b200 import binding
from oracle import decoder, init, rollout, sampler, philox

DEV = "cuda:0"


def oracle_shape(d):
    return decoder.Shape(**{k: d[k] for k in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn",
                                              "vocab", "rope_base", "rms_eps", "dtype")})


def make_ctx(shape_dict, n_groups, G, max_prefix, max_new, chunk=None, extra_blocks=0):
    blocks = n_groups * (-(-max_prefix // 16)) + n_groups * G * (-(-max_new // 16)) + extra_blocks + 8
    chunk = chunk or max(max_prefix, G * max_new) * 2
    return rpo.Context(binding.shape_from_dict(shape_dict), blocks, max_groups=n_groups + 2, max_seqs=n_groups * G,
                       max_chunk_tokens=chunk, max_positions=max_prefix + max_new + 1)


def dev_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(DEV)


def run_decode(ctx, groups, G, S, smp, forced=None, want_logits=False):
    B = len(groups) * G
    V = ctx.shape.vocab
    toks = torch.full((B, S), -7, dtype=torch.int32, device=DEV)
    lens = torch.full((B,), -7, dtype=torch.int32, device=DEV)
    lps = torch.full((B, S), 7.0, dtype=torch.float32, device=DEV)
    dbg = torch.zeros((B, S, V), dtype=torch.float32, device=DEV) if want_logits else None
    ctx.decode_suffix(groups, G, S, smp, toks, lens, lps, d_forced_tokens=None if forced is None else dev_i32(forced),
                      d_logits_dbg=dbg)
    torch.cuda.synchronize()
    return toks.cpu().numpy(), lens.cpu().numpy(), lps.cpu().numpy(), (dbg.cpu().numpy() if want_logits else None)


def oracle_tokens_from_logits(logits, smp, group_ids, G, lens):
    """Apply the oracle's sampler to given float32 logits [B,S,V] with the Philox draws of (seq, step)."""
    B, S, _ = logits.shape
    out = np.zeros((B, S), dtype=np.int32)
    for b in range(B):
        seq = int(group_ids[b // G]) * G + b % G
        for j in range(int(lens[b])):
            if smp.greedy:
                out[b, j] = sampler.greedy_token(logits[b, j])
            else:
                u = int(philox.sampler_u24(smp.seed, seq, j))
                out[b, j] = sampler.sample_token(logits[b, j], smp.temperature, smp.top_p, u)
        out[b, int(lens[b]):] = smp.eos_id
    return out
