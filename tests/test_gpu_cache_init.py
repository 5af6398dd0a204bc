"""Cache initialisation with continuous batching on the GPU: the responses do not depend on the
batch size (random streams are keyed by request and wave), finished sequences free their slots."""
import numpy as np
import pytest

import paper_2601_19404_b200 as rpo
from paper_2601_19404_b200 import cache_init, experience
import workloads
from gpu_util import make_ctx

pytestmark = pytest.mark.gpu

SHAPE = dict(n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=32, rope_base=10000.0,
             rms_eps=1e-6, dtype="fp32")


def test_continuous_batching_fills_the_cache_independently_of_the_batch_size():
    EOS, WAVE, MAX_LEN = 5, 8, 48
    lens = np.array([9, 30, 4, 17, 12, 25, 6], dtype=np.int32)
    toks, off = workloads.prefix_tokens(lens, SHAPE["vocab"], seed=11)
    questions = {100 + k: toks[off[k]:off[k + 1]] for k in range(len(lens))}
    smp = rpo.Sampler(1.0, 1.0, False, EOS, 3)
    results = []
    for mb in (2, 7):
        with make_ctx(SHAPE, mb, 1, int(lens.max()) + MAX_LEN, WAVE) as ctx:
            ctx.init_weights(seed=0, std=0.02)
            cache = experience.ExperienceCache()
            st = cache_init.initialise_cache(cache, ctx, smp, questions, mb, WAVE, MAX_LEN)
            assert ctx.device_status() == 0 and ctx.counters()[1] == ctx.limits.kv_pool_blocks   # every block returned
            assert len(cache) == len(questions) and st["useful_tokens"] <= st["slot_tokens"]
            results.append({q: cache.retrieve(q)[1] for q in questions})
    a, b = results
    sizes = []
    for q in questions:
        assert np.array_equal(a[q], b[q])
        r = a[q]
        assert 1 <= r.size <= MAX_LEN and (r[-1] == EOS or r.size == MAX_LEN) and EOS not in r[:-1]
        sizes.append(r.size)
    assert len(set(sizes)) > 1 and min(sizes) < MAX_LEN          # with 32 tokens and T = 1, EOS comes up at varied lengths


def test_every_cached_response_equals_the_oracle_run_wave_by_wave():
    """The cache the library fills (Section 3.1, Eq. 1) against the oracle: the same scheduler drives
    `oracle.rollout` wave by wave with the same (request, wave) stream ids, on the float32 decoder,
    and every response must come out token for token."""
    from oracle import decoder, init, rollout
    EOS, WAVE, MAX_LEN, MB = 5, 8, 40, 3
    lens = np.array([9, 21, 4, 17, 12], dtype=np.int32)
    toks, off = workloads.prefix_tokens(lens, SHAPE["vocab"], seed=13)
    prompts = [toks[off[k]:off[k + 1]] for k in range(len(lens))]
    sh = decoder.Shape(**SHAPE)
    w = init.init_weights(sh, seed=0, std=0.02)
    ocfg = rollout.SamplerCfg(1.0, 1.0, False, 3, EOS)

    def oracle_engine(prefixes, group_ids, max_new):
        outs = [rollout.rollout_group(w, sh, p, 1, max_new, ocfg, group_id=int(g)) for p, g in zip(prefixes, group_ids)]
        return np.stack([o["tokens"][0] for o in outs]), np.array([o["lens"][0] for o in outs], dtype=np.int32)

    want, want_stats = cache_init.schedule(prompts, oracle_engine, MB, WAVE, MAX_LEN, EOS)
    with make_ctx(SHAPE, MB, 1, int(lens.max()) + MAX_LEN, WAVE) as ctx:
        ctx.init_weights(seed=0, std=0.02)
        got, got_stats = cache_init.schedule(prompts, cache_init.library_engine(ctx, rpo.Sampler(1.0, 1.0, False, EOS, 3)),
                                             MB, WAVE, MAX_LEN, EOS)
        assert ctx.device_status() == 0
    assert got_stats == want_stats
    for r in range(len(prompts)):
        assert np.array_equal(got[r], want[r]), r
    assert len({g.size for g in got}) > 1
