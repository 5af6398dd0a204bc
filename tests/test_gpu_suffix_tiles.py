"""Decode attention over long private suffixes against the oracle, element by element.

The decode attention deals the 64-key tiles of a sequence's own suffix round-robin over the
prefix splits of its group (tile j of sequence i goes to split (i + j) mod n_splits) and merges the
splits' partial results.  These cases make that index arithmetic matter: suffixes of several
tiles per sequence, ragged prefixes long enough for several splits, groups with more suffix tiles
than splits and groups with fewer, sequences that stop at an EOS in the middle of a tile, and the
shape of a full-path rollout (a short prompt, hundreds of generated tokens).  All floating-point
comparisons are teacher-forced and use the stated bf16 tolerances (logits 3e-2, log-probs 2e-2)."""
import numpy as np
import pytest
import torch

import paper_2601_19404_b200 as rpo
import workloads
from oracle import exactmath as em, init, rollout
from gpu_util import DEV, oracle_shape, make_ctx, dev_i32, run_decode

pytestmark = pytest.mark.gpu

SHAPE = dict(n_layers=4, d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=128, d_ffn=1536, vocab=4096,
             rope_base=1e6, rms_eps=1e-6, dtype="bf16")


def _forced_with_stops(n_seq, S, vocab, eos, stops, seed):
    """Teacher tokens without the EOS id, except at the given (sequence -> position) stops."""
    forced = workloads.teacher_tokens(n_seq, S, vocab, seed=seed)
    forced[forced == eos] = eos + 1
    for b, j in stops.items():
        forced[b, j] = eos
    return forced


def _check_against_oracle(sh_d, w, lens, G, S, forced, eos, stops, fast=1, scale_qk=None, tol=(3e-2, 2e-2)):
    sh = oracle_shape(sh_d)
    n_g = len(lens)
    with make_ctx(sh_d, n_g, G, int(lens.max()), S, chunk=max(2048, int(lens.max()))) as ctx:
        ctx.set_option("use_tcgen05", min(fast, 1)); ctx.set_option("use_tc_attention", min(fast, 1))
        ctx.set_option("use_fused_layers", 2 if fast == 2 else 1)      # 2: fused GEMM epilogues forced
        ctx.set_option("use_tc5_decode", 1 if fast == 3 else 0)        # 3: the tcgen05 decode attention
        ctx.set_option("use_tc5_pipelined", 1 if fast == 4 else 0)     # 4: the pipelined tcgen05 attention in prefill / log-prob passes
        ctx.init_weights(0, 0.02)
        if scale_qk is not None:                       # sharper attention: the same scaled q/k weights on both sides
            for l in range(sh.n_layers):
                for n in ("wq", "wk"):
                    ctx.write_tensor(f"layers.{l}.{n}", em.to_bf16_bits(w[f"layers.{l}.{n}"]))
        toks, off = workloads.prefix_tokens(lens, sh.vocab, seed=12)
        groups = ctx.prefill_prefix(dev_i32(toks), off)
        smp = rpo.Sampler(1.0, 0.95, False, eos, 0)
        t, l, lp, dbg = run_decode(ctx, groups, G, S, smp, forced=forced, want_logits=True)
        # lengths and the padding after a stop
        for b in range(n_g * G):
            n = stops.get(b, S - 1) + 1
            assert l[b] == n and np.array_equal(t[b, :n], forced[b, :n])
            assert np.all(t[b, n:] == eos) and np.all(lp[b, n:] == 0.0)
        pol = torch.zeros((n_g * G, S), dtype=torch.float32, device=DEV)
        ctx.token_logprobs(groups, G, S, dev_i32(t), dev_i32(l), pol)
        torch.cuda.synchronize()
        pol = pol.cpu().numpy()
        if fast >= 1:
            # the same pass with the output head that keeps (max, sum of exponentials, target logit) per tile instead of
            # writing the logits: forced here, since this vocabulary is too small for it to be chosen
            ctx.set_option("use_fused_lse", 2)
            pol2 = torch.zeros((n_g * G, S), dtype=torch.float32, device=DEV)
            ctx.token_logprobs(groups, G, S, dev_i32(t), dev_i32(l), pol2)
            torch.cuda.synchronize()
            pol2 = pol2.cpu().numpy()
            assert np.array_equal(pol2 == 0.0, pol == 0.0) and float(np.max(np.abs(pol2 - pol))) <= 2e-5
            pol = pol2                                # the comparison with the oracle below runs on the fused result
        worst = [0.0, 0.0, 0.0]
        for g in range(n_g):
            sl = slice(g * G, (g + 1) * G)
            ref_lp, ref_logits = rollout.token_logprobs(w, sh, toks[off[g]:off[g + 1]], t[sl], l[sl], want_logits=True)
            for i in range(G):
                n = int(l[g * G + i])
                err = np.abs(dbg[g * G + i, :n] - ref_logits[i])
                worst[0] = max(worst[0], float(err.max()))
                srt = np.sort(ref_logits[i], axis=-1)
                clear = (srt[:, -1] - srt[:, -2]) > 0.05
                assert np.all((np.argmax(dbg[g * G + i, :n], -1) == np.argmax(ref_logits[i], -1))[clear])
            worst[1] = max(worst[1], float(np.max(np.abs(lp[sl] - ref_lp))))
            worst[2] = max(worst[2], float(np.max(np.abs(pol[sl] - ref_lp))))
        assert worst[0] <= tol[0] and worst[1] <= tol[1] and worst[2] <= tol[1], worst
        assert ctx.device_status() == 0
        ctx.release_groups(groups)
        assert ctx.counters()[1] == ctx.limits.kv_pool_blocks
        return worst


@pytest.mark.parametrize("fast", [4, 3, 2, 1, 0], ids=["tcgen05_pipelined_prefill_attention", "tcgen05_decode_attention", "tensor_core_fused_epilogues",
                                                       "tensor_core_kernels", "cuda_core_kernels"])
def test_ragged_long_prefixes_and_multi_tile_suffixes_with_stops(fast):
    """Prefixes of 1100 / 37 / 650 tokens (several prefix splits for the long ones, none for the
    short one), G = 6, 230 suffix tokens = 4 key tiles per sequence; stops inside the first tile, on a
    tile boundary and inside the third tile."""
    sh = oracle_shape(SHAPE)
    w = init.init_weights(sh, seed=0, std=0.02)
    lens = np.array([1100, 37, 650], dtype=np.int32)
    G, S, eos = 6, 230, 7
    stops = {1: 20, 4: 63, 5: 64, 8: 150, 13: 128, 16: 229}
    forced = _forced_with_stops(len(lens) * G, S, sh.vocab, eos, stops, seed=31)
    _check_against_oracle(SHAPE, w, lens, G, S, forced, eos, stops, fast=fast)


def test_full_path_shape_short_prompt_long_generation():
    """The shape of a full-path rollout (no cached reasoning prefix): a 17-token prompt, G = 8, 300
    generated tokens, so the private suffix (5 key tiles) carries almost all of the attention."""
    sh = oracle_shape(SHAPE)
    w = init.init_weights(sh, seed=0, std=0.02)
    lens = np.array([17, 17], dtype=np.int32)
    G, S, eos = 8, 300, 7
    stops = {3: 290, 9: 70}
    forced = _forced_with_stops(len(lens) * G, S, sh.vocab, eos, stops, seed=32)
    for fast in (4, 3, 2, 1):
        _check_against_oracle(SHAPE, w, lens, G, S, forced, eos, stops, fast=fast)


def test_sharp_attention_makes_single_keys_matter():
    """With N(0, 0.02) weights the attention is nearly uniform and one mis-masked key among hundreds
    would hide in the rounding noise.  Here the q and k projections are scaled by 3, which puts most of
    a row's weight on a few keys, so every key's visibility shows in the logits.  The scores are nine
    times larger and so is their rounding error; the tolerances are scaled accordingly and the float32
    CUDA-core path has to land in the same place."""
    sh = oracle_shape(SHAPE)
    w = init.init_weights(sh, seed=0, std=0.02)
    for l in range(sh.n_layers):
        for n in ("wq", "wk"):
            w[f"layers.{l}.{n}"] = em.round_bf16((w[f"layers.{l}.{n}"] * np.float32(3.0)).astype(np.float32))
    lens = np.array([700, 90], dtype=np.int32)
    G, S, eos = 4, 140, 7
    stops = {2: 100}
    forced = _forced_with_stops(len(lens) * G, S, sh.vocab, eos, stops, seed=33)
    worst = {f: _check_against_oracle(SHAPE, w, lens, G, S, forced, eos, stops, fast=f, scale_qk=3.0, tol=(9e-2, 6e-2))
             for f in (4, 3, 2, 1, 0)}
    assert all(worst[f][0] <= 1.5 * worst[0][0] + 5e-3 for f in (1, 2, 3, 4)), worst
