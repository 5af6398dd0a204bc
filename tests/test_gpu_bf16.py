"""bf16 parity on a small decoder: logits max-abs <= 3e-2, log-probs <= 2e-2 (teacher-forced),
greedy argmax equal where the oracle's top-2 gap exceeds 0.05, sampler decisions exact."""
import numpy as np
import pytest
import torch

import paper_2601_19404_b200 as rpo
import workloads
from oracle import init, rollout
from gpu_util import DEV, oracle_shape, make_ctx, dev_i32, run_decode, oracle_tokens_from_logits

pytestmark = pytest.mark.gpu

SHAPES = {
    "dh128": dict(n_layers=4, d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=128, d_ffn=1536, vocab=4096,
                  rope_base=1e6, rms_eps=1e-6, dtype="bf16"),
    "dh64": dict(n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=4, head_dim=64, d_ffn=688, vocab=1000,
                 rope_base=1e4, rms_eps=1e-6, dtype="bf16"),
}


@pytest.mark.parametrize("name", list(SHAPES))
@pytest.mark.parametrize("fast", [0, 1, 2], ids=["cuda_core_kernels", "tensor_core_kernels", "tensor_core_fused_epilogues"])
def test_bf16_small_decoder_parity(name, fast):
    sh_d = SHAPES[name]
    sh = oracle_shape(sh_d)
    w = init.init_weights(sh, seed=0, std=0.02)
    lens = np.array([200, 37, 129], dtype=np.int32)
    G, S = 4, 21
    with make_ctx(sh_d, len(lens), G, int(lens.max()), S, chunk=256) as ctx:
        # 2: RMSNorm / RoPE / KV append / SwiGLU / residual as GEMM epilogues even where the planner would
        # keep the separate kernels (many thin split-K planes at these small sizes)
        ctx.set_option("use_tcgen05", min(fast, 1)); ctx.set_option("use_tc_attention", min(fast, 1))
        ctx.set_option("use_fused_layers", 2 if fast == 2 else 1)
        ctx.init_weights(0, 0.02)
        toks, off = workloads.prefix_tokens(lens, sh.vocab, seed=2)
        groups = ctx.prefill_prefix(dev_i32(toks), off)
        forced = workloads.teacher_tokens(len(lens) * G, S, sh.vocab, seed=8)
        t, l, lp, dbg = run_decode(ctx, groups, G, S, rpo.Sampler(1.0, 0.95, False, -1, 0), forced=forced, want_logits=True)
        gaps_ok = total = 0
        for g in range(len(lens)):
            ref = rollout.rollout_group(w, sh, toks[off[g]:off[g + 1]], G, S, rollout.SamplerCfg(1.0, 0.95), group_id=g,
                                        forced_tokens=forced[g * G:(g + 1) * G], want_logits=True)
            sl = slice(g * G, (g + 1) * G)
            assert np.max(np.abs(dbg[sl] - ref["logits"])) <= 3e-2
            assert np.max(np.abs(lp[sl] - ref["logprobs"])) <= 2e-2
            srt = np.sort(ref["logits"], axis=-1)
            clear = (srt[..., -1] - srt[..., -2]) > 0.05
            agree = np.argmax(dbg[sl], -1) == np.argmax(ref["logits"], -1)
            assert np.all(agree[clear])
            gaps_ok += int(clear.sum()); total += clear.size
        # sampled run: decisions are exactly the oracle sampler's on the GPU's own float32 logits
        smp = rpo.Sampler(1.0, 0.95, False, -1, 123)
        t, l, lp, dbg = run_decode(ctx, groups, G, S, smp, want_logits=True)
        assert np.array_equal(t, oracle_tokens_from_logits(dbg, rollout.SamplerCfg(1.0, 0.95, False, 123), range(len(lens)), G, l))
        out = torch.zeros((len(lens) * G, S), dtype=torch.float32, device=DEV)
        ctx.token_logprobs(groups, G, S, dev_i32(t), dev_i32(l), out)
        torch.cuda.synchronize()
        for g in range(len(lens)):
            ref = rollout.token_logprobs(w, sh, toks[off[g]:off[g + 1]], t[g * G:(g + 1) * G], l[g * G:(g + 1) * G])
            assert np.max(np.abs(out.cpu().numpy()[g * G:(g + 1) * G] - ref)) <= 2e-2
        assert ctx.device_status() == 0


@pytest.mark.parametrize("name", list(SHAPES))
def test_in_cluster_merge_equals_merge_kernel(name):
    """Decode attention: merging the prefix splits inside a thread-block cluster (distributed shared
    memory) gives the same logits, bit for bit, as partials in global memory + the merge kernel;
    ragged prefixes, so some splits of the short groups hold suffix tiles only or nothing."""
    sh_d = SHAPES[name]
    lens = np.array([200, 37, 129, 64], dtype=np.int32)
    G, S = 4, 70                                    # suffixes longer than one key tile
    forced = workloads.teacher_tokens(len(lens) * G, S, sh_d["vocab"], seed=9)
    outs = []
    for cl in (1, 0):
        with make_ctx(sh_d, len(lens), G, int(lens.max()), S, chunk=256) as ctx:
            ctx.set_option("use_cluster_merge", cl)
            ctx.init_weights(0, 0.02)
            toks, off = workloads.prefix_tokens(lens, sh_d["vocab"], seed=2)
            groups = ctx.prefill_prefix(dev_i32(toks), off)
            t, l, lp, dbg = run_decode(ctx, groups, G, S, rpo.Sampler(1.0, 0.95, False, -1, 0), forced=forced, want_logits=True)
            assert ctx.device_status() == 0
            outs.append((dbg, lp))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
