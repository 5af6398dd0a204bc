"""Pins for the sampler, log-probabilities and the group rollout of the oracle."""
import math
from fractions import Fraction
import numpy as np
import torch
from oracle import sampler, rollout, decoder, init, philox, exactmath as em

RNG = np.random.default_rng(21)


def exact_top_p24(top_p):
    """floor(float32(top_p) * 2^24) in exact rational arithmetic (no call of the code under test)."""
    return math.floor(Fraction(float(np.float32(top_p))) * (1 << 24))


def test_top_p_fixed_point_is_the_exact_floor():
    for tp in [0.0, 1.0, 0.5, 0.9, 0.95, 0.3, 1e-9, 2.0 ** -24, 2.0 ** -25, 1.0 - 2.0 ** -24, 0.1, 1 / 3, 0.999999]:
        assert sampler.top_p_fixed(tp) == exact_top_p24(tp), tp
    assert sampler.top_p_fixed(0.95) == 15938355 and sampler.top_p_fixed(0.9) == 15099494   # float32(0.95), float32(0.9)
    assert sampler.top_p_fixed(1.0) == 1 << 24 and sampler.top_p_fixed(0.0) == 0
    for tp in RNG.uniform(0, 1, 200):
        assert sampler.top_p_fixed(tp) == exact_top_p24(tp)


def brute_sample(w, top_p, u24):
    """Sort-based textbook nucleus on integer weights with python ints."""
    w = [int(x) for x in w]
    total = sum(w)
    target = (total * exact_top_p24(top_p)) >> 24
    order = sorted(range(len(w)), key=lambda i: -w[i])
    acc, n = 0, 0
    while True:                                   # smallest sorted prefix reaching the target ...
        acc += w[order[n]]; n += 1
        if acc >= target:
            break
    while n < len(w) and w[order[n]] == w[order[n - 1]]:   # ... extended through ties
        acc += w[order[n]]; n += 1
    members = sorted(order[:n])
    r = (acc * u24) >> 24
    run = 0
    for i in members:
        run += w[i]
        if run > r:
            return i, set(members), acc
    raise AssertionError("no token selected")


def test_sampler_equals_sorted_brute_force_on_small_vocabularies():
    for trial in range(300):
        V = int(RNG.integers(2, 9))
        logits = (RNG.standard_normal(V) * RNG.choice([0.1, 1.0, 4.0])).astype(np.float32)
        if trial % 3 == 0:
            logits[RNG.integers(0, V)] = logits[RNG.integers(0, V)]        # force ties
        T = float(RNG.choice([0.5, 0.7, 1.0, 1.5])); top_p = float(RNG.choice([0.0, 0.3, 0.9, 0.95, 1.0]))
        w = sampler.quantised_weights(logits, T)
        for u24 in list(range(0, 1 << 24, 1 << 17)) + [(1 << 24) - 1]:
            tok, members, mass = brute_sample(w, top_p, u24)
            assert sampler.sample_token(logits, T, top_p, u24) == tok
        tau, m = sampler.nucleus_threshold(w, top_p)
        assert m == mass and {i for i in range(V) if w[i] >= tau} == members


def test_quantised_weights_follow_softmax():
    logits = (RNG.standard_normal(500) * 2).astype(np.float32)
    w = sampler.quantised_weights(logits, 0.7).astype(np.float64)
    p = torch.softmax(torch.from_numpy(logits.astype(np.float64)) / 0.7, 0).numpy()
    assert np.max(np.abs(w / w.sum() - p)) < 1e-6      # float32 z = logit/T and float32 exp
    assert w.max() == 2.0 ** 30                                 # the maximum maps to exactly 2^30
    far = np.array([0.0, -30.0], dtype=np.float32)
    assert sampler.quantised_weights(far, 1.0).tolist() == [2 ** 30, 0]


def test_nucleus_mass_is_sufficient_and_minimal():
    for _ in range(50):
        logits = (RNG.standard_normal(2000) * 1.5).astype(np.float32)
        top_p = float(RNG.uniform(0.05, 0.99))
        w = sampler.quantised_weights(logits, 1.0)
        tau, mass = sampler.nucleus_threshold(w, top_p)
        total = int(w.sum()); target = (total * exact_top_p24(top_p)) >> 24
        assert mass >= target
        assert mass - int(w[w == tau].sum()) < target          # dropping the tie class at tau falls short


def test_limits_top_p_one_zero_and_cold_temperature():
    logits = (RNG.standard_normal(64)).astype(np.float32)
    w = sampler.quantised_weights(logits, 1.0)
    tau, mass = sampler.nucleus_threshold(w, 1.0)
    assert mass == int(w.sum())                                  # top_p = 1: plain categorical
    for u24 in (0, 12345, (1 << 24) - 1):
        assert sampler.sample_token(logits, 1.0, 0.0, u24) == sampler.greedy_token(logits)
        assert sampler.sample_token(logits, 1e-3, 0.9, u24) == sampler.greedy_token(logits)
    tie = np.array([1.0, 3.0, 3.0, 2.0], dtype=np.float32)
    assert sampler.greedy_token(tie) == 1                        # lowest id among maxima


def test_categorical_frequencies_chi_square():
    V = 16
    logits = (RNG.standard_normal(V)).astype(np.float32)
    n = 100000
    u = philox.sampler_u24(seed=77, seq=np.arange(n), step=3)
    w = sampler.quantised_weights(logits, 1.0)
    # top_p = 1: vectorised inverse CDF identical to sample_token's definition
    run = np.cumsum(w.astype(np.uint64))
    r = (int(run[-1]) * u.astype(object)) >> 24
    toks = np.searchsorted(run.astype(np.float64), np.array(r, dtype=np.float64), side="right")
    for i in range(0, n, 9973):
        assert sampler.sample_token(logits, 1.0, 1.0, int(u[i])) == toks[i]
    p = torch.softmax(torch.from_numpy(logits.astype(np.float64)), 0).numpy()
    counts = np.bincount(toks, minlength=V)
    chi2 = float(((counts - n * p) ** 2 / (n * p)).sum())
    assert chi2 < 45.0                                            # 15 dof, p ~ 1e-4


def test_log_softmax_library_and_normalisation():
    logits = (RNG.standard_normal(300) * 3).astype(np.float32)
    ours = sampler.log_softmax_row(logits, 0.7)
    ref = torch.log_softmax(torch.from_numpy(logits.astype(np.float64)) / 0.7, 0).numpy()
    assert np.allclose(ours, ref, atol=1e-12)
    assert abs(np.exp(ours).sum() - 1) < 1e-12
    assert sampler.token_logprob(logits, 0.7, 5) == ours[5]


def _model():
    sh = decoder.Shape(2, 32, 4, 2, 8, 48, 64)
    return sh, init.init_weights(sh, 1, 0.25)


def test_rollout_determinism_streams_and_logprob_consistency():
    sh, w = _model()
    prefix = RNG.integers(0, 64, 10)
    cfg = rollout.SamplerCfg(temperature=0.8, top_p=0.9, seed=5)
    a = rollout.rollout_group(w, sh, prefix, G=4, max_new=6, cfg=cfg, group_id=2, want_logits=True)
    b = rollout.rollout_group(w, sh, prefix, G=4, max_new=6, cfg=cfg, group_id=2)
    assert np.array_equal(a["tokens"], b["tokens"]) and np.array_equal(a["logprobs"], b["logprobs"])
    c = rollout.rollout_group(w, sh, prefix, 4, 6, rollout.SamplerCfg(0.8, 0.9, seed=6), group_id=2)
    assert not np.array_equal(a["tokens"], c["tokens"])
    # all G samples draw step 0 from the same logits vector
    assert all(np.array_equal(a["logits"][0, 0], a["logits"][i, 0]) for i in range(4))
    # the draw of sample i at step j uses sequence number group_id*G + i
    u = int(philox.sampler_u24(5, 2 * 4 + 3, 0))
    assert a["tokens"][3, 0] == sampler.sample_token(a["logits"][3, 0], 0.8, 0.9, u)
    # decode-time log-probs == teacher-forced log-probs == full recompute of the whole string
    lp = rollout.token_logprobs(w, sh, prefix, a["tokens"], a["lens"], inv_temperature=1 / 0.8)
    assert np.allclose(lp, a["logprobs"], atol=1e-9)
    i = 1
    full = decoder.forward_full(w, sh, np.concatenate([prefix, a["tokens"][i]]))
    ref = [sampler.log_softmax_row(full[len(prefix) - 1 + j].astype(np.float32), 0.8)[a["tokens"][i, j]] for j in range(6)]
    assert np.allclose(ref, a["logprobs"][i], atol=1e-6)
    assert abs(sum(ref) - a["logprobs"][i].sum()) < 1e-5          # sequence log-likelihood


def test_rollout_greedy_eos_and_forced_tokens():
    sh, w = _model()
    prefix = RNG.integers(0, 64, 7)
    g = rollout.rollout_group(w, sh, prefix, 2, 8, rollout.SamplerCfg(greedy=True), want_logits=True)
    assert np.array_equal(g["tokens"][0], g["tokens"][1])        # greedy: all samples coincide
    assert g["tokens"][0, 0] == int(np.argmax(g["logits"][0, 0]))
    eos = int(g["tokens"][0, 3])                                  # a token greedy emits mid-sequence
    first = int(np.argmax(g["tokens"][0] == eos))
    e = rollout.rollout_group(w, sh, prefix, 2, 8, rollout.SamplerCfg(greedy=True, eos_id=eos))
    assert e["lens"].tolist() == [first + 1] * 2
    assert np.all(e["tokens"][:, first:] == eos) and np.all(e["logprobs"][:, first + 1:] == 0)
    assert e["logprobs"][0, first] < 0 and np.array_equal(e["tokens"][:, :first + 1], g["tokens"][:, :first + 1])
    forced = RNG.integers(0, 64, (2, 8))
    f = rollout.rollout_group(w, sh, prefix, 2, 8, rollout.SamplerCfg(), forced_tokens=forced, want_logits=True)
    assert np.array_equal(f["tokens"], forced)
    full = decoder.forward_full(w, sh, np.concatenate([prefix, forced[1]]))
    assert np.allclose(f["logits"][1], full[6:-1], atol=1e-5)
