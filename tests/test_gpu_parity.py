"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle."""
import numpy as np
import pytest
import torch

import paper_2601_19404_b200 as rpo
from paper_2601_19404_b200 import binding
import workloads
from oracle import decoder, init, rollout, sampler, philox, exactmath as em
from gpu_util import DEV, oracle_shape, make_ctx, dev_i32, run_decode, oracle_tokens_from_logits

pytestmark = pytest.mark.gpu

TINY = workloads.SHAPES["tiny"]
SMALL_BF16 = dict(n_layers=3, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=128, d_ffn=512, vocab=2048,
                  rope_base=1e6, rms_eps=1e-6, dtype="bf16")


@pytest.mark.parametrize("shape", [TINY, SMALL_BF16], ids=["tiny_fp32", "small_bf16"])
def test_init_weights_bit_exact(shape):
    sh = oracle_shape(shape)
    with make_ctx(shape, 1, 1, 32, 4) as ctx:
        ctx.init_weights(seed=1234567890123, std=0.02)
        ref = init.init_weights(sh, seed=1234567890123, std=0.02)
        for name, want in ref.items():
            got = ctx.read_tensor(name)
            if got.dtype == np.uint16:
                assert np.array_equal(got, em.to_bf16_bits(want)), name
            else:
                assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), name
        assert ctx.device_status() == 0


def test_sampler_rows_bit_exact_against_oracle():
    with make_ctx(TINY, 1, 1, 32, 4) as ctx:
        cases = [(6, 1024, 1.0, False, 1.0, 0.9), (4, 1024, 3.0, True, 0.7, 0.95), (3, 151936, 0.78, False, 1.0, 0.95),
                 (2, 151936, 0.78, True, 1.0, 0.95), (3, 5000, 6.0, False, 1.3, 0.5), (2, 1000, 1.0, False, 1.0, 1.0),
                 (2, 1000, 1.0, False, 1.0, 0.0), (2, 33, 1.0, False, 0.5, 0.9)]
        for ci, (n, V, sigma, ties, T, top_p) in enumerate(cases):
            logits = workloads.logits_rows(n, V, sigma, seed=ci, bf16_like=ties)
            seqs = np.arange(n, dtype=np.int64) * 7 + (1 << 33)
            d_logits = torch.from_numpy(logits).to(DEV)
            d_seq = torch.from_numpy(seqs).to(DEV)
            for step in (0, 5):
                smp = rpo.Sampler(T, top_p, False, -1, seed=99 + ci)
                toks = torch.zeros(n, dtype=torch.int32, device=DEV); lps = torch.zeros(n, dtype=torch.float32, device=DEV)
                ctx.sample_rows(d_logits, smp, d_seq, step, toks, lps)
                torch.cuda.synchronize()
                toks = toks.cpu().numpy(); lps = lps.cpu().numpy()
                for r in range(n):
                    u = int(philox.sampler_u24(99 + ci, int(seqs[r]), step))
                    want = sampler.sample_token(logits[r], T, top_p, u)
                    assert toks[r] == want, (ci, r, step)
                    assert abs(lps[r] - sampler.token_logprob(logits[r], T, want)) < 1e-4
            g = rpo.Sampler(T, top_p, True, -1, 0)
            toks = torch.zeros(n, dtype=torch.int32, device=DEV)
            ctx.sample_rows(d_logits, g, d_seq, 0, toks)
            torch.cuda.synchronize()
            assert toks.cpu().tolist() == [sampler.greedy_token(l) for l in logits]


@pytest.mark.parametrize("shape,tol", [(TINY, 2e-5), (SMALL_BF16, 2e-5)], ids=["fp32", "bf16"])
def test_cuda_core_gemm_against_numpy(shape, tol):
    rng = np.random.default_rng(0)
    with make_ctx(shape, 1, 1, 32, 4) as ctx:
        for (M, N, K) in [(1, 8, 8), (37, 100, 72), (130, 257, 688), (64, 64, 16)]:
            a = rng.standard_normal((M, K)).astype(np.float32); w = rng.standard_normal((N, K)).astype(np.float32)
            if shape["dtype"] == "bf16":
                a = em.round_bf16(a); w = em.round_bf16(w)
                dA = torch.from_numpy(a).to(DEV).to(torch.bfloat16); dW = torch.from_numpy(w).to(DEV).to(torch.bfloat16)
            else:
                dA = torch.from_numpy(a).to(DEV); dW = torch.from_numpy(w).to(DEV)
            dC = torch.zeros((M, N), dtype=torch.float32, device=DEV)
            ctx.gemm(dA, dW, dC, impl=1)
            torch.cuda.synchronize()
            ref = a.astype(np.float64) @ w.astype(np.float64).T
            assert np.max(np.abs(dC.cpu().numpy() - ref)) < tol * K ** 0.5 * 4


def _prefill(ctx, lens, vocab, seed=0, group_ids=None):
    toks, off = workloads.prefix_tokens(np.asarray(lens, dtype=np.int32), vocab, seed)
    groups = ctx.prefill_prefix(dev_i32(toks), off, group_ids)
    return toks, off, groups


def test_config1_tiny_fp32_full_parity():
    """Config 1: 2 groups x G=4, prefix 128, suffix 32, greedy and top-p 0.9 at T=1."""
    cfg = workloads.CONFIGS["cfg1_tiny"]
    sh = oracle_shape(TINY)
    w = init.init_weights(sh, seed=0, std=0.02)
    G, S, n_g = cfg["G"], cfg["suffix"], cfg["n_groups"]
    lens = workloads.prefix_lengths(cfg)
    with make_ctx(TINY, n_g, G, int(lens.max()), S) as ctx:
        ctx.init_weights(seed=0, std=0.02)
        toks, off, groups = _prefill(ctx, lens, sh.vocab)
        # --- teacher-forced logits on tokens that come from the input generator
        forced = workloads.teacher_tokens(n_g * G, S, sh.vocab, seed=3)
        t, l, lp, dbg = run_decode(ctx, groups, G, S, rpo.Sampler(1.0, 0.9, False, -1, 0), forced=forced, want_logits=True)
        assert np.array_equal(t, forced) and np.all(l == S)
        for g in range(n_g):
            ref = rollout.rollout_group(w, sh, toks[off[g]:off[g + 1]], G, S, rollout.SamplerCfg(1.0, 0.9), group_id=g,
                                        forced_tokens=forced[g * G:(g + 1) * G], want_logits=True)
            assert np.max(np.abs(dbg[g * G:(g + 1) * G] - ref["logits"])) < 1e-4
            assert np.max(np.abs(lp[g * G:(g + 1) * G] - ref["logprobs"])) < 1e-4
        # --- sampled run: tokens are exactly the oracle sampler's decision on the logits the GPU drew from
        for smp, cfg_o in [(rpo.Sampler(1.0, 0.9, False, -1, 0), rollout.SamplerCfg(1.0, 0.9, False, 0)),
                           (rpo.Sampler(1.0, 1.0, True, -1, 0), rollout.SamplerCfg(1.0, 1.0, True, 0))]:
            t, l, lp, dbg = run_decode(ctx, groups, G, S, smp, want_logits=True)
            assert np.all(l == S)
            assert np.array_equal(t, oracle_tokens_from_logits(dbg, cfg_o, [0, 1], G, l))
            # independent end-to-end oracle rollout: identical tokens while the trajectories agree
            same = 0
            for g in range(n_g):
                ref = rollout.rollout_group(w, sh, toks[off[g]:off[g + 1]], G, S, cfg_o, group_id=g, want_logits=True)
                for i in range(G):
                    b = g * G + i
                    n_same = S if np.array_equal(t[b], ref["tokens"][i]) else int(np.argmax(t[b] != ref["tokens"][i]))
                    same += n_same
                    # up to the first divergence the logits and log-probs must agree
                    assert np.max(np.abs(dbg[b, :n_same + 1] - ref["logits"][i, :n_same + 1])) < 1e-4 if n_same < S else True
                    assert np.max(np.abs(lp[b, :n_same] - ref["logprobs"][i, :n_same])) < 1e-4 if n_same else True
                    if cfg_o.greedy and n_same < S:      # a greedy mismatch is only allowed at a near tie
                        top2 = np.sort(ref["logits"][i, n_same])[-2:]
                        assert top2[1] - top2[0] <= 0.05
            assert same >= 0.9 * n_g * G * S
        # --- determinism: same seed, same bytes
        t2, l2, lp2, _ = run_decode(ctx, groups, G, S, rpo.Sampler(1.0, 0.9, False, -1, 0))
        t3, l3, lp3, _ = run_decode(ctx, groups, G, S, rpo.Sampler(1.0, 0.9, False, -1, 0))
        assert np.array_equal(t2, t3) and np.array_equal(lp2.view(np.uint32), lp3.view(np.uint32))
        # --- token log-probs of the sampled suffixes (Eq. 7), teacher-forced
        out = torch.zeros((n_g * G, S), dtype=torch.float32, device=DEV)
        ctx.token_logprobs(groups, G, S, dev_i32(t2), dev_i32(l2), out)
        torch.cuda.synchronize()
        assert np.max(np.abs(out.cpu().numpy() - lp2)) < 1e-4       # decode-time == teacher-forced
        for g in range(n_g):
            ref = rollout.token_logprobs(w, sh, toks[off[g]:off[g + 1]], t2[g * G:(g + 1) * G], l2[g * G:(g + 1) * G])
            assert np.max(np.abs(out.cpu().numpy()[g * G:(g + 1) * G] - ref)) < 1e-4
        assert ctx.device_status() == 0
        ctx.release_groups(groups)


def test_ragged_prefixes_gains_eos_and_group_ids():
    """Ragged prefix lengths around the 16-token block size, non-unit gains, EOS stop, custom ids."""
    sh_d = dict(TINY, n_layers=2, vocab=512)
    sh = oracle_shape(sh_d)
    rng = np.random.default_rng(5)
    w = init.init_weights(sh, seed=7, std=0.05)
    lens = [1, 15, 16, 17, 33, 50]
    G, S = 3, 19
    gids = [11, 3, 0, 250, 9, 4]
    with make_ctx(sh_d, len(lens), G, max(lens), S, chunk=64) as ctx:        # chunk 64 forces several prefill passes
        ctx.init_weights(seed=7, std=0.05)
        for name in ["gf"] + [f"layers.{l}.{g}" for l in range(2) for g in ("g1", "g2")]:
            w[name] = (1.0 + 0.2 * rng.standard_normal(sh.d_model)).astype(np.float32)
            ctx.write_tensor(name, w[name])
        toks, off, groups = _prefill(ctx, lens, sh.vocab, seed=1, group_ids=gids)
        assert [g.prefix_len for g in groups] == lens and [g.group_id for g in groups] == gids
        greedy = rpo.Sampler(1.0, 1.0, True, -1, 0)
        t, l, lp, dbg = run_decode(ctx, groups, G, S, greedy, want_logits=True)
        refs = [rollout.rollout_group(w, sh, toks[off[g]:off[g + 1]], G, S, rollout.SamplerCfg(greedy=True), group_id=gids[g],
                                      want_logits=True) for g in range(len(lens))]
        for g, ref in enumerate(refs):
            assert np.max(np.abs(dbg[g * G, 0] - ref["logits"][0, 0])) < 1e-4       # step-0 logits (prefill parity)
        # EOS: a token the oracle's greedy run emits mid-sequence in group 2
        eos = int(refs[2]["tokens"][0, 6])
        smp = rpo.Sampler(0.9, 0.95, False, eos, 42)
        t, l, lp, dbg = run_decode(ctx, groups, G, S, smp, want_logits=True)
        cfg_o = rollout.SamplerCfg(0.9, 0.95, False, 42, eos)
        assert np.array_equal(t, oracle_tokens_from_logits(dbg, cfg_o, gids, G, l))
        for b in range(len(lens) * G):
            n = int(l[b])
            hits = np.nonzero(t[b] == eos)[0]
            assert n == (hits[0] + 1 if hits.size else S)
            assert np.all(t[b, n:] == eos) and np.all(lp[b, n:] == 0.0) and np.all(lp[b, :n] < 0)
        # teacher-force the GPU's own tokens through the oracle: logits at every live position
        for g in range(len(lens)):
            ref = rollout.rollout_group(w, sh, toks[off[g]:off[g + 1]], G, S, cfg_o, group_id=gids[g],
                                        forced_tokens=t[g * G:(g + 1) * G], want_logits=True)
            for i in range(G):
                n = int(l[g * G + i])
                assert n == ref["lens"][i]
                assert np.max(np.abs(dbg[g * G + i, :n] - ref["logits"][i, :n])) < 1e-4
                assert np.max(np.abs(lp[g * G + i, :n] - ref["logprobs"][i, :n])) < 1e-4
        out = torch.full((len(lens) * G, S), 5.0, dtype=torch.float32, device=DEV)
        ctx.token_logprobs(groups, G, S, dev_i32(t), dev_i32(l), out, inv_temperature=1 / 0.9)
        torch.cuda.synchronize()
        assert np.max(np.abs(out.cpu().numpy() - lp)) < 1e-4
        assert ctx.device_status() == 0


def test_shared_prefix_equals_private_prefix_and_block_accounting():
    sh_d = dict(TINY, vocab=256)
    G, S, P = 4, 9, 40
    with make_ctx(sh_d, 5, G, P, S) as ctx:
        ctx.init_weights(seed=2, std=0.05)
        _, free0 = ctx.counters()
        toks, off = workloads.prefix_tokens(np.array([P], dtype=np.int32), 256, seed=9)
        shared = ctx.prefill_prefix(dev_i32(toks), off, [6])
        forced = workloads.teacher_tokens(G, S, 256, seed=1)
        _, _, lp_s, dbg_s = run_decode(ctx, shared, G, S, rpo.Sampler(), forced=forced, want_logits=True)
        # the same prefix prefilled four times, one private copy per sample
        toks4 = np.tile(toks, G); off4 = np.arange(G + 1, dtype=np.int32) * P
        private = ctx.prefill_prefix(dev_i32(toks4), off4, [6 * G + i for i in range(G)])
        _, free1 = ctx.counters()
        assert free0 - free1 == 5 * 3                                        # ceil(40/16) blocks per prefill
        _, _, lp_p, dbg_p = run_decode(ctx, private, 1, S, rpo.Sampler(), forced=forced, want_logits=True)
        assert np.max(np.abs(dbg_s - dbg_p)) < 2e-5 and np.max(np.abs(lp_s - lp_p)) < 2e-5
        # sampled: sequence numbers coincide (6*G+i), so the tokens must too
        smp = rpo.Sampler(1.0, 0.9, False, -1, 5)
        t_s, _, _, _ = run_decode(ctx, shared, G, S, smp)
        t_p, _, _, _ = run_decode(ctx, private, 1, S, smp)
        assert np.array_equal(t_s, t_p)
        ctx.release_groups(shared); ctx.release_groups(private)
        assert ctx.counters()[1] == free0


def test_errors_limits_and_edge_sizes():
    sh_d = dict(TINY, vocab=128)
    ctx = rpo.Context(binding.shape_from_dict(sh_d), kv_pool_blocks=6, max_groups=2, max_seqs=4, max_chunk_tokens=64,
                      max_positions=80)
    toks = dev_i32(np.arange(64) % 128)
    with pytest.raises(rpo.RpoError) as e:
        ctx.prefill_prefix(toks, [0, 10])
    assert e.value.code == -6                                                # weights not initialised
    ctx.init_weights(0, 0.02)
    with pytest.raises(rpo.RpoError) as e:
        ctx.prefill_prefix(toks, [0, 0])
    assert e.value.code == -1                                                # empty prefix
    with pytest.raises(rpo.RpoError) as e:
        ctx.prefill_prefix(dev_i32(np.zeros(200)), [0, 70])
    assert e.value.code == -7                                                # longer than a chunk
    g = ctx.prefill_prefix(toks, [0, 64])                                    # 4 blocks of 6
    with pytest.raises(rpo.RpoError) as e:
        ctx.prefill_prefix(toks, [0, 64])
    assert e.value.code == -3 and ctx.counters()[1] == 2                    # pool exhausted, nothing leaked
    out = torch.zeros(4 * 40, dtype=torch.int32, device=DEV); lens = torch.zeros(4, dtype=torch.int32, device=DEV)
    with pytest.raises(rpo.RpoError) as e:
        ctx.decode_suffix(g, 8, 4, rpo.Sampler(), out, lens)
    assert e.value.code == -7                                                # B > max_seqs
    with pytest.raises(rpo.RpoError) as e:
        ctx.decode_suffix(g, 4, 17, rpo.Sampler(), out, lens)
    assert e.value.code == -7                                                # positions
    with pytest.raises(rpo.RpoError) as e:
        ctx.decode_suffix(g, 4, 16, rpo.Sampler(temperature=0.0), out, lens)
    assert e.value.code == -1
    with pytest.raises(rpo.RpoError) as e:
        ctx.decode_suffix(g, 4, 16, rpo.Sampler(), out, lens)                # needs 4 private blocks, 2 free
    assert e.value.code == -3 and ctx.counters()[1] == 2
    ctx.decode_suffix(g, 2, 16, rpo.Sampler(), out, lens)                    # exactly fits
    ctx.decode_suffix(g, 1, 1, rpo.Sampler(), out, lens)                     # single step: step-0 draw only
    torch.cuda.synchronize()
    assert lens.cpu().tolist()[:1] == [1] and ctx.counters()[1] == 2
    ctx.release_groups(g)
    with pytest.raises(rpo.RpoError) as e:
        ctx.decode_suffix(g, 1, 1, rpo.Sampler(), out, lens)
    assert e.value.code == -6                                                # stale handle
    bad = ctx.prefill_prefix(dev_i32(np.array([5, 9999, -3, 7])), [0, 4])    # out-of-range ids: clamped + flagged
    assert ctx.device_status() == 2 and ctx.device_status() == 0
    ctx.release_groups(bad)
    ctx.close()


def test_rollout_host_matches_device_calls():
    sh_d = dict(TINY, vocab=300)
    G, S = 2, 7
    lens = np.array([20, 9, 31], dtype=np.int32)
    with make_ctx(sh_d, 3, G, 31, S) as ctx:
        ctx.init_weights(3, 0.05)
        toks, off = workloads.prefix_tokens(lens, 300, seed=4)
        smp = rpo.Sampler(0.8, 0.9, False, -1, 17)
        groups = ctx.prefill_prefix(dev_i32(toks), off)
        t, l, lp, _ = run_decode(ctx, groups, G, S, smp)
        ctx.release_groups(groups)
        ht = np.zeros((3 * G, S), dtype=np.int32); hl = np.zeros(3 * G, dtype=np.int32)
        hp = np.zeros((3 * G, S), dtype=np.float32); hq = np.zeros((3 * G, S), dtype=np.float32)
        ctx.rollout_host(toks, off, G, S, smp, ht, hl, hp, hq)
        assert np.array_equal(ht, t) and np.array_equal(hl, l) and np.array_equal(hp, lp)
        assert np.max(np.abs(hq - hp)) < 1e-4
        assert ctx.counters()[1] == ctx.limits.kv_pool_blocks
        # the context keeps its device staging between calls: a smaller call, then the first one again
        # (same addresses, so the decode step's graph is reused), give the same answers
        t2, off2 = toks[:off[2]], off[:3]
        h2 = np.zeros((2 * G, S), dtype=np.int32); l2 = np.zeros(2 * G, dtype=np.int32); p2 = np.zeros((2 * G, S), dtype=np.float32)
        ctx.rollout_host(t2, off2, G, S, smp, h2, l2, p2, None)
        assert np.array_equal(h2, t[:2 * G]) and np.array_equal(l2, l[:2 * G]) and np.array_equal(p2, lp[:2 * G])
        ht[:] = 0; hp[:] = 0
        ctx.rollout_host(toks, off, G, S, smp, ht, hl, hp, hq)
        assert np.array_equal(ht, t) and np.array_equal(hp, lp)
        assert ctx.counters()[1] == ctx.limits.kv_pool_blocks and ctx.device_status() == 0


def test_tensor_core_gemm_against_numpy():
    """tcgen05/TMA GEMM (bf16 in, float32 accumulate) on shapes spanning several tiles, ragged M/N
    tails, every tile width and a deep K."""
    rng = np.random.default_rng(3)
    shape = dict(SMALL_BF16)
    with make_ctx(shape, 1, 1, 32, 4) as ctx:
        for (M, N, K) in [(128, 256, 64), (1, 16, 64), (12, 48, 128), (129, 272, 192), (300, 4096, 512),
                          (128, 2048, 1536), (40, 1536, 8960), (1000, 512, 256), (257, 2384, 128)]:
            a = em.round_bf16((rng.standard_normal((M, K))).astype(np.float32))
            w = em.round_bf16((rng.standard_normal((N, K)) * 0.05).astype(np.float32))
            dA = torch.from_numpy(a).to(DEV).to(torch.bfloat16); dW = torch.from_numpy(w).to(DEV).to(torch.bfloat16)
            dC = torch.full((M, N), 777.0, dtype=torch.float32, device=DEV)
            ref = a.astype(np.float64) @ w.astype(np.float64).T
            for bn in (0, 512, 384):                 # the planner's kernel, then CTA-pair tiles of 256 and of 128 rows
                ctx.set_option("gemm_bn", bn)
                dC.fill_(777.0)
                ctx.gemm(dA, dW, dC, impl=2)
                torch.cuda.synchronize()
                assert ctx.device_status() == 0
                err = np.max(np.abs(dC.cpu().numpy() - ref))
                assert err < 2e-5 * K ** 0.5, (M, N, K, bn, err)
            ctx.set_option("gemm_bn", 0)
        with pytest.raises(rpo.RpoError):
            ctx.gemm(torch.zeros((8, 72), dtype=torch.bfloat16, device=DEV), torch.zeros((16, 72), dtype=torch.bfloat16, device=DEV),
                     torch.zeros((8, 16), dtype=torch.float32, device=DEV), impl=2)      # K % 64 != 0


def _sampled_gemm_error(dA, dW, dC, n_samples, rng):
    """max |C - A W^T| over randomly sampled outputs, the reference dot products in float64 on the host."""
    M, K = dA.shape
    N = dW.shape[0]
    mi = rng.integers(0, M, n_samples); ni = rng.integers(0, N, n_samples)
    a = dA[torch.from_numpy(mi).to(DEV)].float().cpu().numpy().astype(np.float64)
    w = dW[torch.from_numpy(ni).to(DEV)].float().cpu().numpy().astype(np.float64)
    ref = np.einsum("ik,ik->i", a, w)
    got = dC[torch.from_numpy(mi).to(DEV), torch.from_numpy(ni).to(DEV)].cpu().numpy()
    return float(np.max(np.abs(got - ref)))


@pytest.mark.parametrize("M,N,K", [(128, 17920, 1536), (256, 152064, 3584), (512, 1536, 8960), (4096, 4608, 3584)],
                         ids=["decode_gate_up_1p5b", "decode_lm_head_7b", "decode_down_1p5b_B512", "prefill_qkv_7b"])
def test_tensor_core_gemm_full_size_every_tile_width_and_split(M, N, K):
    """The GEMM at the sizes the benchmark configurations launch it with, for every tile width and
    several split-K factors the planner may choose (many work items per persistent CTA), checked on
    sampled outputs, plus the planner's own choice."""
    rng = np.random.default_rng(11)
    shape = dict(SMALL_BF16)
    gen = torch.Generator(device=DEV); gen.manual_seed(5)
    dA = torch.randn((M, K), device=DEV, generator=gen).to(torch.bfloat16)
    dW = (torch.randn((N, K), device=DEV, generator=gen) * 0.05).to(torch.bfloat16)
    with make_ctx(shape, 1, 1, 32, 4) as ctx:
        for bn, splits in [(0, 0), (512, 1), (512, 3), (384, 1), (384, 2), (256, 1), (128, 1), (96, 1), (64, 1), (32, 1), (128, 4), (64, 3), (256, 2)]:   # 512 / 384 = CTA-pair tiles with 128 / 64 rows per CTA
            ctx.set_option("gemm_bn", bn); ctx.set_option("gemm_splits", splits)
            dC = torch.full((M, N), 777.0, dtype=torch.float32, device=DEV)
            ctx.gemm(dA, dW, dC, impl=2)
            torch.cuda.synchronize()
            assert ctx.device_status() == 0
            err = _sampled_gemm_error(dA, dW, dC, 4000, rng)
            assert err < 2e-5 * K ** 0.5, (bn, splits, err)
            # edges of the output: first/last rows and columns are written
            assert float(dC[0, 0]) != 777.0 and float(dC[M - 1, N - 1]) != 777.0 and float(dC[M - 1, 0]) != 777.0
            del dC
