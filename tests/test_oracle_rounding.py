"""Pins for the oracle's optional storage rounding (`decoder.Rounding`).

The rounding mode is a model of a bf16 implementation, not the definition, so the pins
are about its relation to the definition: switched off it IS the definition bit for
bit; every switch on its own moves the result, rounds exactly the tensor it names and
nothing else, and stays within the distance bf16 storage is allowed to cost on shallow
decoders (logits 3e-2, log-probs 2e-2)."""
import dataclasses

import numpy as np
import pytest

from oracle import decoder, exactmath as em, init, rollout

RNG = np.random.default_rng(23)
ALL_ON = decoder.Rounding(norm="gain", qkv=False, q=True, kv=True, p=True, attn_out=True, act=True, trig_f32=True)
SWITCHES = [dict(norm="normalised"), dict(norm="gain"), dict(qkv=True), dict(q=True), dict(kv=True), dict(p=True),
            dict(attn_out=True), dict(act=True), dict(trig_f32=True)]


def shape(n_layers=2, dtype="bf16", **over):
    kw = dict(n_layers=n_layers, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ffn=96, vocab=128,
              rope_base=10000.0, rms_eps=1e-6, dtype=dtype)
    kw.update(over)
    return decoder.Shape(**kw)


def weights(sh, seed=0, std=0.1):
    w = init.init_weights(sh, seed, std)
    for k in list(w):                     # gains away from 1 so that "x * g" and "x" round differently
        if k.endswith(("g1", "g2")) or k == "gf":
            w[k] = (1.0 + 0.3 * RNG.standard_normal(w[k].shape)).astype(np.float32)
    return w


def representable(x):
    x32 = np.asarray(x).astype(np.float32)
    return np.array_equal(em.round_bf16(x32), x32) and np.array_equal(x32.astype(np.asarray(x).dtype), x)


def test_all_switches_off_is_the_definition_bit_for_bit():
    sh = shape()
    w = weights(sh)
    toks = RNG.integers(0, sh.vocab, 19)
    plain = decoder.forward_full(w, sh, toks)
    assert np.array_equal(plain, decoder.forward_full(w, sh, toks, rnd=decoder.Rounding()))
    sp0, sp1 = decoder.SharedPrefix(w, sh, toks[:11]), decoder.SharedPrefix(w, sh, toks[:11], rnd=decoder.Rounding())
    assert np.array_equal(sp0.teacher_forced_logits(toks[11:]), sp1.teacher_forced_logits(toks[11:]))
    i0, i1 = decoder.Incremental(w, sh), decoder.Incremental(w, sh, rnd=decoder.Rounding())
    for t in toks[:5]:
        assert np.array_equal(i0.step(t), i1.step(t))
    cfg = rollout.SamplerCfg(1.0, 0.9, False, 3, -1)
    a = rollout.rollout_group(w, sh, toks[:11], 3, 6, cfg, want_logits=True)
    b = rollout.rollout_group(w, sh, toks[:11], 3, 6, cfg, want_logits=True, rnd=decoder.Rounding())
    assert all(np.array_equal(a[k], b[k]) for k in a)


@pytest.mark.parametrize("switch", SWITCHES, ids=lambda s: "+".join(f"{k}={v}" for k, v in s.items()))
def test_each_switch_alone_moves_the_result_a_little(switch):
    sh = shape()
    w = weights(sh)
    toks = RNG.integers(0, sh.vocab, 40)
    plain = decoder.forward_full(w, sh, toks)
    moved = decoder.forward_full(w, sh, toks, rnd=decoder.Rounding(**switch))
    err = np.max(np.abs(moved - plain))
    assert err > 0.0                                           # the switch does something ...
    limit = 1e-5 if "trig_f32" in switch else 3e-2
    assert err < limit                                         # ... of the size of one 16-bit (or float32) rounding


def test_rounded_tensors_are_exactly_the_named_ones():
    sh = shape(n_layers=1)
    w = weights(sh)
    x = RNG.standard_normal((5, sh.d_model))
    pos = np.arange(5) + 3
    # q / kv: the rotated tensors come out bf16-representable, the others untouched
    q0, k0, v0 = decoder._qkv(w, sh, 0, x, pos, np.float64, decoder.Rounding())
    q1, k1, v1 = decoder._qkv(w, sh, 0, x, pos, np.float64, decoder.Rounding(q=True))
    assert representable(q1) and np.array_equal(q1, decoder._bf16(q0)) and np.array_equal(k1, k0) and np.array_equal(v1, v0)
    q2, k2, v2 = decoder._qkv(w, sh, 0, x, pos, np.float64, decoder.Rounding(kv=True))
    assert np.array_equal(q2, q0) and np.array_equal(k2, decoder._bf16(k0)) and np.array_equal(v2, decoder._bf16(v0))
    assert not representable(q0) and not representable(k0)
    # qkv: rounded BEFORE the rotation, so the rotated values are in general not representable
    q3, k3, v3 = decoder._qkv(w, sh, 0, x, pos, np.float64, decoder.Rounding(qkv=True))
    assert representable(v3) and not representable(q3)
    unrot = decoder.rope(q3, -pos.astype(np.float64), sh.rope_base)      # rotating back recovers the rounded projection
    assert np.max(np.abs(unrot - decoder._bf16(unrot))) < 1e-12
    # attn_out / p
    vis = np.tril(np.ones((5, 5), dtype=bool))
    a0 = decoder.attend(q0, k0, v0, vis)
    assert np.array_equal(decoder.attend(q0, k0, v0, vis, decoder.Rounding(attn_out=True)), decoder._bf16(a0))
    ap = decoder.attend(q0, k0, v0, vis, decoder.Rounding(p=True))
    assert 0 < np.max(np.abs(ap - a0)) < 4e-3 * np.max(np.abs(v0))       # each weight off by < 2^-8 relative
    # row 0 sees one key: its only probability is exp(0) = 1, representable, so nothing moves
    assert np.allclose(ap[0], a0[0], rtol=0, atol=1e-15)


def test_norm_modes_against_their_formulas():
    d = 48
    x = RNG.standard_normal((7, d)) * 3.0
    g = 1.0 + 0.3 * RNG.standard_normal(d)
    W = RNG.standard_normal((11, d))
    inv = 1.0 / np.sqrt((x * x).mean(-1, keepdims=True) + 1e-6)
    bf = lambda a: em.round_bf16(a.astype(np.float32)).astype(np.float64)
    off, = decoder.normed_products(x, g, 1e-6, [W], decoder.Rounding())
    nrm, = decoder.normed_products(x, g, 1e-6, [W], decoder.Rounding(norm="normalised"))
    gain, = decoder.normed_products(x, g, 1e-6, [W], decoder.Rounding(norm="gain"))
    assert np.allclose(off, (x * inv * g) @ W.T, rtol=0, atol=1e-12)
    assert np.allclose(nrm, bf(x * inv * g) @ W.T, rtol=0, atol=1e-12)
    assert np.allclose(gain, (bf(x * g) @ W.T) * inv, rtol=0, atol=1e-12)
    # both rounded variants are one bf16 rounding of the input away from the definition
    scale = np.abs(x * inv * g) @ np.abs(W).T
    assert np.all(np.abs(nrm - off) <= 2.0 ** -8 * scale) and np.all(np.abs(gain - off) <= 2.0 ** -8 * scale)
    assert not np.array_equal(nrm, gain)
    # "gain" with g = 1 on an input that is already representable rounds nothing
    xb = bf(x)
    a, = decoder.normed_products(xb, np.ones(d), 1e-6, [W], decoder.Rounding(norm="gain"))
    b, = decoder.normed_products(xb, np.ones(d), 1e-6, [W], decoder.Rounding())
    assert np.allclose(a, b, rtol=0, atol=1e-12)
    with pytest.raises(ValueError):
        decoder.Rounding(norm="sometimes")


@pytest.mark.parametrize("n_layers", [2, 4])
def test_all_switches_on_stays_within_the_bf16_budget_on_shallow_decoders(n_layers):
    """Storage rounding costs at most the stated bf16 tolerances (logits 3e-2, log-probs 2e-2) on
    decoders of up to four layers with N(0, 0.02) weights, for both norm placements."""
    sh = shape(n_layers=n_layers, d_model=128, n_q_heads=4, n_kv_heads=2, head_dim=32, d_ffn=256, vocab=512)
    w = init.init_weights(sh, 0, 0.02)
    toks = RNG.integers(0, sh.vocab, 90)
    forced = RNG.integers(0, sh.vocab, (3, 12))
    cfg = rollout.SamplerCfg(1.0, 0.95)
    ref = rollout.rollout_group(w, sh, toks, 3, 12, cfg, forced_tokens=forced, want_logits=True)
    for norm in ("normalised", "gain"):
        rnd = dataclasses.replace(ALL_ON, norm=norm)
        got = rollout.rollout_group(w, sh, toks, 3, 12, cfg, forced_tokens=forced, want_logits=True, rnd=rnd)
        assert 0 < np.max(np.abs(got["logits"] - ref["logits"])) <= 3e-2
        assert np.max(np.abs(got["logprobs"] - ref["logprobs"])) <= 2e-2


def test_rounded_variants_of_the_three_routines_agree():
    """Incremental decode, shared-prefix decode and the dense recompute round the same tensors, so
    with rounding on they still agree to float64 accuracy (the P rounding acts on exp(s - max) over
    the same visible keys in all three)."""
    sh = shape()
    w = weights(sh)
    toks = RNG.integers(0, sh.vocab, 23)
    full = decoder.forward_full(w, sh, toks, rnd=ALL_ON)
    inc = decoder.Incremental(w, sh, rnd=ALL_ON)
    steps = np.stack([inc.step(t) for t in toks])
    assert np.max(np.abs(steps - full)) < 1e-9
    sp = decoder.SharedPrefix(w, sh, toks[:14], rnd=ALL_ON)
    tf = sp.teacher_forced_logits(toks[14:])           # row j: distribution of token 14 + j
    assert np.max(np.abs(tf - full[13:22])) < 1e-9
