"""Pins for the oracle's decoder forward: library routines, closed forms, invariants
and a pure-Python brute force, so that a dropped term, a wrong sign or index, or a
transposed operand anywhere in `oracle.decoder` fails at least one test."""
import math
import numpy as np
import pytest
import torch
import torch.nn.functional as tF
from oracle import decoder, init

RNG = np.random.default_rng(11)


def small(dtype="fp32", **over):
    kw = dict(n_layers=2, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ffn=48, vocab=64,
              rope_base=10000.0, rms_eps=1e-6, dtype=dtype)
    kw.update(over)
    return decoder.Shape(**kw)


def weights(sh, seed=0, std=0.3):
    w = init.init_weights(sh, seed, std)
    for k in list(w):                     # non-trivial gains so that g1/g2/gf mix-ups show
        if k.endswith(("g1", "g2")) or k == "gf":
            w[k] = (1.0 + 0.3 * RNG.standard_normal(w[k].shape)).astype(np.float32)
    return w


def test_rmsnorm_library_and_invariants():
    x = RNG.standard_normal((5, 32)); g = RNG.standard_normal(32)
    ours = decoder.rmsnorm(x, g, 1e-6)
    ref = tF.rms_norm(torch.from_numpy(x), (32,), torch.from_numpy(g), 1e-6).numpy()
    assert np.allclose(ours, ref, atol=1e-12)
    y = decoder.rmsnorm(x, np.ones(32), 0.0)
    assert np.allclose(np.sqrt((y * y).mean(-1)), 1.0)
    assert np.allclose(decoder.rmsnorm(7.5 * x, g, 0.0), decoder.rmsnorm(x, g, 0.0))
    assert np.allclose(decoder.rmsnorm(np.full((1, 4), 2.0), np.ones(4), 5.0), 2.0 / 3.0)   # eps inside the root


def test_rope_properties():
    x = RNG.standard_normal((6, 3, 8)); y = RNG.standard_normal((6, 3, 8))
    pos = np.array([0, 1, 5, 17, 100, 4000])
    rx = decoder.rope(x, pos, 10000.0)
    assert np.allclose(np.linalg.norm(rx, axis=-1), np.linalg.norm(x, axis=-1))
    assert np.allclose(rx[0], x[0])                                  # position 0 is the identity
    # q_m . k_n depends only on m - n
    a = decoder.rope(x[:1], [9], 1e4)[0, 0] @ decoder.rope(y[:1], [4], 1e4)[0, 0]
    b = decoder.rope(x[:1], [1009], 1e4)[0, 0] @ decoder.rope(y[:1], [1004], 1e4)[0, 0]
    assert abs(a - b) < 1e-9
    # explicit rotate-half pairing (i, i + dh/2) with theta_i = base^(-2i/dh)
    v = np.zeros((1, 1, 8)); v[0, 0, 1] = 1.0
    out = decoder.rope(v, [3], 100.0)[0, 0]
    th = 3 * 100.0 ** (-2 * 1 / 8)
    expect = np.zeros(8); expect[1] = math.cos(th); expect[5] = math.sin(th)
    assert np.allclose(out, expect)


def test_attention_against_library_and_closed_forms():
    T, hq, hkv, dh = 7, 4, 2, 8
    q = RNG.standard_normal((T, hq, dh)); k = RNG.standard_normal((T, hkv, dh)); v = RNG.standard_normal((T, hkv, dh))
    causal = np.tril(np.ones((T, T), dtype=bool))
    ours = decoder.attend(q, k, v, causal)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(2, dim=0)[None]   # kv head h//2 for q head h
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(2, dim=0)[None]
    ref = tF.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.allclose(ours, ref, atol=1e-12)
    one = decoder.attend(q[:1], k[:1], v[:1], np.ones((1, 1), dtype=bool))
    assert np.allclose(one[0, 0], v[0, 0]) and np.allclose(one[0, 3], v[0, 1])
    same_k = np.repeat(k[:1], T, axis=0)
    mean = decoder.attend(q, same_k, v, np.ones((T, T), dtype=bool))
    assert np.allclose(mean[2, 1], v[:, 0].mean(0))


def test_silu_library():
    x = RNG.standard_normal(100) * 4
    assert np.allclose(decoder.silu(x), tF.silu(torch.from_numpy(x)).numpy(), atol=1e-13)


def brute_forward(w, sh, tokens):
    """Pure-Python scalar loops, written from the formulas, no numpy linear algebra."""
    d, hq, hkv, dh, F_, V = sh.d_model, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.d_ffn, sh.vocab
    W = {k: np.asarray(v, dtype=np.float64).tolist() for k, v in w.items()}

    def norm(x, g):
        ms = sum(a * a for a in x) / len(x)
        return [a / math.sqrt(ms + sh.rms_eps) * gg for a, gg in zip(x, g)]

    def lin(x, M):                                     # y_o = sum_i M[o][i] x_i
        return [sum(M[o][i] * x[i] for i in range(len(x))) for o in range(len(M))]

    def rot(vec, pos):
        out = list(vec)
        for i in range(dh // 2):
            th = pos * sh.rope_base ** (-2.0 * i / dh)
            a, b = vec[i], vec[i + dh // 2]
            out[i] = a * math.cos(th) - b * math.sin(th)
            out[i + dh // 2] = b * math.cos(th) + a * math.sin(th)
        return out

    xs = [list(W["embed"][t]) for t in tokens]
    for l in range(sh.n_layers):
        p = f"layers.{l}."
        qs, ks, vs = [], [], []
        for t, x in enumerate(xs):
            h = norm(x, W[p + "g1"])
            q, k, v = lin(h, W[p + "wq"]), lin(h, W[p + "wk"]), lin(h, W[p + "wv"])
            qs.append([rot(q[i * dh:(i + 1) * dh], t) for i in range(hq)])
            ks.append([rot(k[i * dh:(i + 1) * dh], t) for i in range(hkv)])
            vs.append([v[i * dh:(i + 1) * dh] for i in range(hkv)])
        new = []
        for t, x in enumerate(xs):
            a = []
            for i in range(hq):
                j = i // (hq // hkv)
                sc = [sum(qs[t][i][c] * ks[u][j][c] for c in range(dh)) / math.sqrt(dh) for u in range(t + 1)]
                m = max(sc); e = [math.exp(s - m) for s in sc]; z = sum(e)
                a += [sum(e[u] / z * vs[u][j][c] for u in range(t + 1)) for c in range(dh)]
            x = [xi + oi for xi, oi in zip(x, lin(a, W[p + "wo"]))]
            h = norm(x, W[p + "g2"])
            g, u_ = lin(h, W[p + "wg"]), lin(h, W[p + "wu"])
            act = [gi / (1 + math.exp(-gi)) * ui for gi, ui in zip(g, u_)]
            new.append([xi + di for xi, di in zip(x, lin(act, W[p + "wd"]))])
        xs = new
    return [lin(norm(x, W["gf"]), W["lm_head"]) for x in xs]


def test_forward_full_equals_scalar_brute_force():
    sh = small(n_layers=2, d_model=12, n_q_heads=4, n_kv_heads=2, head_dim=4, d_ffn=10, vocab=9)
    w = weights(sh, seed=5)
    toks = [3, 8, 0, 3, 5]
    got = decoder.forward_full(w, sh, toks)
    assert np.allclose(got, np.array(brute_forward(w, sh, toks)), atol=1e-10)


def test_zero_layer_closed_form_and_identity_blocks():
    sh = small(n_layers=0)
    w = weights(sh)
    toks = np.array([1, 5, 5, 63])
    e = w["embed"][toks].astype(np.float64)
    expect = decoder.rmsnorm(e, w["gf"].astype(np.float64), sh.rms_eps) @ w["lm_head"].astype(np.float64).T
    assert np.allclose(decoder.forward_full(w, sh, toks), expect)
    sh2 = small(n_layers=2)
    w2 = weights(sh2)
    for l in range(2):                                  # Wo = Wd = 0 -> both residual branches vanish
        w2[f"layers.{l}.wo"][:] = 0; w2[f"layers.{l}.wd"][:] = 0
    e2 = w2["embed"][toks].astype(np.float64)
    expect2 = decoder.rmsnorm(e2, w2["gf"].astype(np.float64), sh2.rms_eps) @ w2["lm_head"].astype(np.float64).T
    assert np.allclose(decoder.forward_full(w2, sh2, toks), expect2)


def test_causality_and_position_shift():
    sh = small(); w = weights(sh)
    toks = RNG.integers(0, 64, 12)
    base = decoder.forward_full(w, sh, toks)
    t2 = toks.copy(); t2[7] = (t2[7] + 1) % 64
    pert = decoder.forward_full(w, sh, t2)
    assert np.allclose(base[:7], pert[:7], atol=1e-12) and not np.allclose(base[7:], pert[7:], atol=1e-6)
    shifted = decoder.forward_full(w, sh, toks, pos0=37)          # RoPE is relative
    assert np.allclose(base, shifted, atol=1e-9)


def test_gqa_equals_mha_with_replicated_kv_heads():
    sh = small(); w = weights(sh)
    mha = small(n_kv_heads=4)
    w2 = dict(w)
    for l in range(2):
        for n in ("wk", "wv"):
            m = w[f"layers.{l}.{n}"].reshape(2, 8, 32)
            w2[f"layers.{l}.{n}"] = np.repeat(m, 2, axis=0).reshape(32, 32)
    toks = RNG.integers(0, 64, 9)
    assert np.allclose(decoder.forward_full(w, sh, toks), decoder.forward_full(w2, mha, toks), atol=1e-11)


def test_incremental_and_shared_prefix_equal_full_recompute():
    sh = small(); w = weights(sh)
    toks = RNG.integers(0, 64, 21)
    full = decoder.forward_full(w, sh, toks)
    inc = decoder.Incremental(w, sh)
    step = np.stack([inc.step(t) for t in toks])
    assert np.allclose(full, step, atol=1e-10)
    P = 13
    sp = decoder.SharedPrefix(w, sh, toks[:P])
    assert np.allclose(sp.step0_logits(), full[P - 1], atol=1e-10)
    tf = sp.teacher_forced_logits(toks[P:])
    assert np.allclose(tf, full[P - 1:-1], atol=1e-10)
    # two different suffixes over one prefix object == two private recomputes
    other = RNG.integers(0, 64, 5)
    tf2 = sp.teacher_forced_logits(other)
    priv = decoder.forward_full(w, sh, np.concatenate([toks[:P], other]))
    assert np.allclose(tf2, priv[P - 1:-1], atol=1e-10)


def test_float32_mode_is_close_to_float64():
    sh = small(); w = weights(sh, std=0.1)
    toks = RNG.integers(0, 64, 16)
    a = decoder.forward_full(w, sh, toks, dt=np.float64)
    b = decoder.forward_full(w, sh, toks, dt=np.float32)
    assert b.dtype == np.float32 and np.max(np.abs(a - b)) < 1e-4


def test_single_layer_routine_chains_to_the_dense_forward():
    """`decoder.layer` (used to check an implementation layer by layer) applied in turn is the dense
    recompute bit for bit, and with a key context it is the shared-prefix routine."""
    sh = small()
    w = weights(sh)
    toks = RNG.integers(0, sh.vocab, 17)
    x = decoder.mat(w, "embed", np.float64)[toks]
    causal = np.tril(np.ones((17, 17), dtype=bool))
    ks, vs = [], []
    for l in range(sh.n_layers):
        x, a, k, v = decoder.layer(w, sh, l, x, np.arange(17), None, None, causal)
        assert a.shape == (17, sh.n_q_heads, sh.head_dim)
        ks.append(k); vs.append(v)
    assert np.array_equal(x, decoder.forward_full(w, sh, toks, return_hidden=True))
    # rows 12.. against a context of the first 12 keys
    x = decoder.mat(w, "embed", np.float64)[toks]
    xs = x[12:]
    vis = np.concatenate([np.ones((5, 12), dtype=bool), np.tril(np.ones((5, 5), dtype=bool))], axis=1)
    hid = decoder.forward_full(w, sh, toks, return_hidden=True)
    for l in range(sh.n_layers):
        xs, _, _, _ = decoder.layer(w, sh, l, xs, np.arange(12, 17), ks[l][:12], vs[l][:12], vis)
    assert np.max(np.abs(xs - hid[12:])) < 1e-12
