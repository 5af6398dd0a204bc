"""rpo_decode_wave: a decode that proceeds in waves and keeps the sequences' private K/V and parked
logits between calls (cache initialisation, Section 3.1, Eq. 1).

What is checked:
  * W calls reproduce ONE rpo_decode_suffix call on the same groups bit for bit (tokens, lengths,
    log-probs), on the float32 CUDA-core path, the tensor-core path and the tcgen05 decode attention,
    with uneven wave sizes that cut KV blocks and key tiles in the middle and sequences that stop at
    an EOS inside a wave;
  * groups at different stages share a call (one joins later, one leaves early): teacher-forced
    log-probs against the oracle within the stated bf16 tolerance;
  * the cache filled through the resumable scheduler equals the oracle's full-path rollout of every
    request, for several batch and wave sizes;
  * reservations: a refused call reserves nothing, releasing a group returns its blocks and rows.
"""
import numpy as np
import pytest
import torch

import paper_2601_19404_b200 as rpo
from paper_2601_19404_b200 import cache_init
import workloads
from oracle import decoder, init, rollout
from gpu_util import DEV, oracle_shape, make_ctx, dev_i32, run_decode

pytestmark = pytest.mark.gpu

TINY = dict(n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=32, rope_base=10000.0,
            rms_eps=1e-6, dtype="fp32")
SMALL = dict(n_layers=4, d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=128, d_ffn=1536, vocab=256,
             rope_base=1e6, rms_eps=1e-6, dtype="bf16")


def _waves(ctx, groups, G, sizes, total, smp, forced=None):
    """Runs the waves; returns (tokens [B, sum(sizes)], lens [B], logprobs) put together from the calls."""
    B = len(groups) * G
    toks, lps, lens, at = [], [], np.zeros(B, dtype=np.int64), 0
    for n in sizes:
        t = torch.full((B, n), -7, dtype=torch.int32, device=DEV)
        l = torch.full((B,), -7, dtype=torch.int32, device=DEV)
        p = torch.full((B, n), 7.0, dtype=torch.float32, device=DEV)
        f = None if forced is None else dev_i32(forced[:, at:at + n])
        ctx.decode_wave(groups, G, n, total, smp, t, l, p, d_forced_tokens=f)
        torch.cuda.synchronize()
        toks.append(t.cpu().numpy()); lps.append(p.cpu().numpy())
        lens += l.cpu().numpy()
        at += n
    return np.concatenate(toks, 1), lens.astype(np.int32), np.concatenate(lps, 1)


@pytest.mark.parametrize("case", ["float32_cuda_cores", "bf16_tensor_cores", "bf16_tcgen05_decode_attention", "bf16_fused_epilogues"])
def test_waves_reproduce_one_decode_call_bit_for_bit(case):
    shape = TINY if case.startswith("float32") else SMALL
    lens = np.array([150, 37, 700] if shape is SMALL else [40, 9, 77], dtype=np.int32)
    G, EOS = 4, 5
    sizes = [5, 16, 1, 42, 70, 22] if shape is SMALL else [3, 16, 1, 20]
    S = sum(sizes)
    per = -(-S // 16)
    with make_ctx(shape, len(lens), G, int(lens.max()), S, extra_blocks=len(lens) * G * per) as ctx:
        if case == "bf16_tcgen05_decode_attention":
            ctx.set_option("use_tc5_decode", 1)
        if case == "bf16_fused_epilogues":
            ctx.set_option("use_fused_layers", 2)
        ctx.init_weights(0, 0.02)
        toks, off = workloads.prefix_tokens(lens, shape["vocab"], seed=21)
        groups = ctx.prefill_prefix(dev_i32(toks), off, np.array([3, 11, 4], dtype=np.int32))
        smp = rpo.Sampler(1.0, 0.98, False, EOS, 17)
        t0, l0, lp0, _ = run_decode(ctx, groups, G, S, smp)
        free_before = ctx.counters()[1]
        t1, l1, lp1 = _waves(ctx, groups, G, sizes, S, smp)
        assert np.array_equal(t1, t0) and np.array_equal(l1, l0)
        assert np.array_equal(lp1.view(np.uint32), lp0.view(np.uint32))
        assert ctx.counters()[1] == free_before - len(lens) * G * per      # the waves' blocks stay with the groups
        assert ctx.device_status() == 0
        ctx.release_groups(groups)
        assert ctx.counters()[1] == ctx.limits.kv_pool_blocks
    stopped = int(np.sum(l0 < S))
    assert 0 < stopped < len(lens) * G, "the case should see sequences that stop and sequences that do not"


def test_groups_at_different_stages_share_a_call_against_the_oracle():
    """Three groups: A and B start together, C joins at the second call, A leaves after the third.  Tokens are
    teacher-forced (with two stops), so every group's log-probs can be compared with the oracle's
    teacher-forced pass over the whole suffix: bf16 tolerance 2e-2."""
    sh = oracle_shape(SMALL)
    w = init.init_weights(sh, seed=0, std=0.02)
    lens = np.array([300, 40, 130], dtype=np.int32)
    G, EOS, S = 3, 5, 60
    forced = workloads.teacher_tokens(3 * G, S, sh.vocab, seed=5)
    forced[forced == EOS] = EOS + 1
    forced[1, 33] = EOS
    forced[7, 16] = EOS
    per = -(-S // 16)
    with make_ctx(SMALL, 3, G, int(lens.max()), S, extra_blocks=3 * G * per) as ctx:
        ctx.init_weights(0, 0.02)
        toks, off = workloads.prefix_tokens(lens, sh.vocab, seed=22)
        groups = ctx.prefill_prefix(dev_i32(toks), off)
        smp = rpo.Sampler(1.0, 0.95, False, EOS, 0)
        Group = type(groups[0])

        def call(members, n, at):
            arr = (Group * len(members))(*[groups[g] for g in members])
            rows = np.concatenate([np.arange(g * G, (g + 1) * G) for g in members])
            f = np.stack([forced[r, at[r // G]:at[r // G] + n] for r in rows])
            t, l, p = _waves(ctx, arr, G, [n], S, smp, forced=f)
            return rows, t, l, p

        got_lp = np.zeros((3 * G, S)); got_len = np.zeros(3 * G, dtype=np.int64)
        at = [0, 0, 0]
        plan = [([0, 1], 16), ([0, 1, 2], 20), ([0, 1, 2], 7), ([1, 2], 17), ([2], 16)]
        for members, n in plan:
            rows, t, l, p = call(members, n, at)
            for k, r in enumerate(rows):
                a = at[r // G]
                got_lp[r, a:a + n] = p[k]; got_len[r] += l[k]
            for g in members:
                at[g] += n
        assert at == [43, 60, 60]
        for g in range(3):
            sl = slice(g * G, (g + 1) * G)
            n = at[g]
            want_len = np.array([min(n, (list(forced[r, :n]).index(EOS) + 1) if EOS in forced[r, :n] else n) for r in range(g * G, (g + 1) * G)])
            assert np.array_equal(got_len[sl], want_len)
            tok = forced[sl, :n].copy()
            ref_lp = rollout.token_logprobs(w, sh, toks[off[g]:off[g + 1]], tok, want_len.astype(np.int32))
            err = max(float(np.max(np.abs(got_lp[g * G + i, :want_len[i]] - ref_lp[i][:want_len[i]]))) for i in range(G))
            assert err <= 2e-2, (g, err)
            for i in range(G):
                assert np.all(got_lp[g * G + i, want_len[i]:n] == 0.0)
        assert ctx.device_status() == 0
        ctx.release_groups(groups)
        assert ctx.counters()[1] == ctx.limits.kv_pool_blocks


def test_resumable_cache_initialisation_equals_the_oracles_full_path_rollouts():
    """Every response of the cache filled wave by wave with kept state (one prefill per request) equals the
    oracle's full-path rollout of that request (Eq. 1) with stream id request * MAX_WAVES, whatever the batch
    size and the wave size."""
    EOS, MAX_LEN = 5, 40
    lens = np.array([9, 21, 4, 17, 12, 30], dtype=np.int32)
    toks, off = workloads.prefix_tokens(lens, TINY["vocab"], seed=13)
    prompts = [toks[off[k]:off[k + 1]] for k in range(len(lens))]
    sh = decoder.Shape(**TINY)
    w = init.init_weights(sh, seed=0, std=0.02)
    ocfg = rollout.SamplerCfg(1.0, 1.0, False, 3, EOS)
    want = []
    for r, p in enumerate(prompts):
        o = rollout.rollout_group(w, sh, p, 1, MAX_LEN, ocfg, group_id=r * cache_init.MAX_WAVES)
        want.append(o["tokens"][0][:int(o["lens"][0])])
    assert len({x.size for x in want}) > 1 and min(x.size for x in want) < MAX_LEN
    for mb, wave in ((3, 8), (2, 5), (6, 40)):
        per = -(-MAX_LEN // 16)
        with make_ctx(TINY, mb, 1, int(lens.max()), MAX_LEN, extra_blocks=mb * per) as ctx:
            ctx.init_weights(seed=0, std=0.02)
            session = cache_init.LibrarySession(ctx, rpo.Sampler(1.0, 1.0, False, EOS, 3), MAX_LEN)
            got, st = cache_init.schedule_resumable(prompts, session, mb, wave, MAX_LEN, EOS)
            assert ctx.device_status() == 0 and ctx.counters()[1] == ctx.limits.kv_pool_blocks and not session.groups
        for r in range(len(prompts)):
            assert np.array_equal(got[r], want[r]), (mb, wave, r)
        assert st["useful_tokens"] == sum(x.size for x in want)


def test_wave_reservations_and_refusals():
    lens = np.array([20, 20], dtype=np.int32)
    with make_ctx(TINY, 2, 2, 20, 32, extra_blocks=0) as ctx:
        ctx.init_weights(0, 0.02)
        toks, off = workloads.prefix_tokens(lens, TINY["vocab"], seed=3)
        groups = ctx.prefill_prefix(dev_i32(toks), off)
        smp = rpo.Sampler(1.0, 1.0, False, -1, 0)
        t = torch.zeros((4, 8), dtype=torch.int32, device=DEV); l = torch.zeros(4, dtype=torch.int32, device=DEV)
        free0 = ctx.counters()[1]
        with pytest.raises(rpo.RpoError) as e:                    # more blocks than the pool has left: nothing is reserved
            ctx.decode_wave(groups, 2, 8, 16 * (free0 + 1), smp, t, l)
        assert e.value.code in (-3, -7) and ctx.counters()[1] == free0
        ctx.decode_wave(groups, 2, 8, 32, smp, t, l)
        assert ctx.counters()[1] == free0 - 2 * 2 * 2
        with pytest.raises(rpo.RpoError) as e:                    # another G than the groups began with
            ctx.decode_wave(groups, 1, 8, 32, smp, t, l)
        assert e.value.code == -7
        ctx.decode_wave(groups, 2, 8, 32, smp, t, l)
        ctx.decode_wave(groups, 2, 8, 32, smp, t, l)
        ctx.decode_wave(groups, 2, 8, 32, smp, t, l)
        with pytest.raises(rpo.RpoError) as e:                    # past the reserved positions
            ctx.decode_wave(groups, 2, 8, 32, smp, t, l)
        assert e.value.code == -7
        # a plain decode call and a log-prob pass on a group in the middle of its waves leave its state alone
        t2 = torch.zeros((4, 5), dtype=torch.int32, device=DEV)
        ctx.decode_suffix(groups, 2, 5, smp, t2, l)
        assert ctx.device_status() == 0
        ctx.release_groups(groups)
        assert ctx.counters()[1] == ctx.limits.kv_pool_blocks
        groups = ctx.prefill_prefix(dev_i32(toks), off)          # state rows came back as well
        ctx.decode_wave(groups, 2, 8, 32, smp, t, l)
        ctx.release_groups(groups)
        assert ctx.device_status() == 0 and ctx.counters()[1] == ctx.limits.kv_pool_blocks
