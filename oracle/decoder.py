"""Plain decoder forward: the function the rollout policy pi_theta evaluates.

The paper names the policy models only; the architecture is the one the benchmark
configurations spell out: pre-norm decoder, RMSNorm (eps inside the root, gains g),
grouped-query attention with rotate-half RoPE, SwiGLU feed-forward, no biases, untied
embedding and output head.  For a token string t_0..t_{n-1}:

    x_t   = E[t_t]
    h     = rmsnorm(x, g1);  q, k, v = h Wq^T, h Wk^T, h Wv^T;  RoPE(q, k; position t)
    s_tu  = q_t . k_u / sqrt(dh) for u <= t, query head i reads kv head i // (Hq/Hkv)
    x    += softmax(s) v Wo^T
    h     = rmsnorm(x, g2);  x += (silu(h Wg^T) * (h Wu^T)) Wd^T
    logits_t = rmsnorm(x_t, gf) W_lm^T

Three routines compute it: `forward_full` (dense recompute, the definition),
`Incremental` (token-by-token with a growing K/V list) and `SharedPrefix` (one K/V of
the cached prefix reused by all G samples of a sampling group, Eq. 3).  The tests pin
the second and third to the first.

Optional storage rounding.  The definition above is what every routine computes when
`rnd` is None.  A 16-bit implementation of the same decoder keeps some intermediate
tensors in bfloat16; `Rounding` names those places one by one, and a routine given a
`Rounding` rounds (to nearest even, through float32) at exactly the places switched
on and nowhere else, all other arithmetic staying in `dt`.  This is a model of a
bf16 implementation used to separate "rounds where it says it rounds" from "computes
something else"; it is not the definition, and with every switch off it is the
definition bit for bit.
"""
from dataclasses import dataclass
import numpy as np
from . import exactmath as em


@dataclass(frozen=True)
class Shape:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-6
    dtype: str = "fp32"          # "fp32" | "bf16": storage type of the matrices


@dataclass(frozen=True)
class Rounding:
    """Places where intermediate values are rounded to bfloat16 (all off = the definition).

    norm     "off" | "normalised" | "gain".  The input of the q/k/v, gate/up and output-head
             products.  "normalised": h = bf16(x / rms(x) * g).  "gain": hb = bf16(x * g) is the
             product's input and each output row is multiplied by 1 / rms(x) afterwards (the row
             scale commutes with the product; only the rounded values differ).
    qkv      the q/k/v projections are rounded before RoPE (an implementation that stores the
             projection and rotates it in a second pass)
    q        the rotated queries are rounded
    kv       the rotated keys and the values are rounded (what a bf16 KV cache holds)
    p        the unnormalised probabilities exp(s - max s) are rounded before they multiply V;
             the row sum that normalises the result is taken over the unrounded values
    attn_out the attention output is rounded (input of the output projection)
    act      silu(gate) * up is rounded (input of the down projection)
    trig_f32 cos / sin of the RoPE angles are rounded to float32 (angles stay float64)
    """
    norm: str = "off"
    qkv: bool = False
    q: bool = False
    kv: bool = False
    p: bool = False
    attn_out: bool = False
    act: bool = False
    trig_f32: bool = False

    def __post_init__(self):
        if self.norm not in ("off", "normalised", "gain"):
            raise ValueError(f"unknown norm rounding {self.norm!r}")


def _bf16(x, on=True):
    """x rounded to bfloat16 (via float32, both to nearest even), in x's dtype; x itself if not on."""
    if not on:
        return x
    return em.round_bf16(np.asarray(x).astype(np.float32)).astype(x.dtype)


def mat(w, name, dt):
    """Matrix `name` as dtype dt (widening compact bf16 bit patterns if needed)."""
    t = w[name]
    if t.dtype == np.uint16:
        t = (t.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return t.astype(dt, copy=False)


def rmsnorm(x, g, eps):
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def rope_angles(pos, head_dim, base):
    """[len(pos), head_dim/2] angles pos * base^(-2i/head_dim), in float64."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    theta = np.float64(base) ** (-2.0 * i / head_dim)
    return np.asarray(pos, dtype=np.float64)[:, None] * theta[None, :]


def rope(x, pos, base, trig_f32=False):
    """Rotate-half RoPE. x: [T, H, dh]; dimension i pairs with i + dh/2."""
    dh = x.shape[-1]
    ang = rope_angles(pos, dh, base)
    c, s = np.cos(ang), np.sin(ang)
    if trig_f32:
        c, s = c.astype(np.float32), s.astype(np.float32)
    c = c[:, None, :].astype(x.dtype)
    s = s[:, None, :].astype(x.dtype)
    x1, x2 = x[..., : dh // 2], x[..., dh // 2:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


def attend(q, k, v, visible, rnd=None):
    """q [T,Hq,dh], k/v [U,Hkv,dh], visible [T,U] bool -> [T,Hq,dh]."""
    T, hq, dh = q.shape
    hkv = k.shape[1]
    rep = hq // hkv
    out = np.empty_like(q)
    scale = 1.0 / np.sqrt(dh)
    for h in range(hq):
        s = (q[:, h, :] @ k[:, h // rep, :].T) * scale
        s = np.where(visible, s, -np.inf)
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s)
        if rnd is not None and rnd.p:
            out[:, h, :] = (_bf16(p) @ v[:, h // rep, :]) / p.sum(axis=-1, keepdims=True)
        else:
            p = p / p.sum(axis=-1, keepdims=True)
            out[:, h, :] = p @ v[:, h // rep, :]
    return _bf16(out, rnd is not None and rnd.attn_out)


def normed_products(x, g, eps, mats, rnd=None):
    """[rmsnorm(x, g) @ W.T for W in mats], with the input rounded as rnd.norm says."""
    if rnd is None or rnd.norm == "off":
        h = rmsnorm(x, g, eps)
        return [h @ W.T for W in mats]
    if rnd.norm == "normalised":
        h = _bf16(rmsnorm(x, g, eps))
        return [h @ W.T for W in mats]
    hb = _bf16(x * g)                                   # "gain": the row scale is applied to the products
    inv = 1.0 / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    return [(hb @ W.T) * inv for W in mats]


def _qkv(w, shape, l, x, pos, dt, rnd=None):
    hq, hkv, dh = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    q, k, v = normed_products(x, mat(w, f"layers.{l}.g1", dt), shape.rms_eps,
                              [mat(w, f"layers.{l}.{n}", dt) for n in ("wq", "wk", "wv")], rnd)
    q, k, v = q.reshape(-1, hq, dh), k.reshape(-1, hkv, dh), v.reshape(-1, hkv, dh)
    if rnd is None:
        return rope(q, pos, shape.rope_base), rope(k, pos, shape.rope_base), v
    q, k, v = _bf16(q, rnd.qkv), _bf16(k, rnd.qkv), _bf16(v, rnd.qkv)
    q = _bf16(rope(q, pos, shape.rope_base, rnd.trig_f32), rnd.q)
    k = _bf16(rope(k, pos, shape.rope_base, rnd.trig_f32), rnd.kv)
    return q, k, _bf16(v, rnd.kv)


def _finish_layer(w, shape, l, x, a, dt, rnd=None):
    x = x + a.reshape(x.shape[0], -1) @ mat(w, f"layers.{l}.wo", dt).T
    gate, up = normed_products(x, mat(w, f"layers.{l}.g2", dt), shape.rms_eps,
                               [mat(w, f"layers.{l}.wg", dt), mat(w, f"layers.{l}.wu", dt)], rnd)
    act = _bf16(silu(gate) * up, rnd is not None and rnd.act)
    return x + act @ mat(w, f"layers.{l}.wd", dt).T


def layer(w, shape, l, x, pos, k_ctx, v_ctx, visible, dt=np.float64, rnd=None):
    """One decoder layer on rows x [T, d] at positions pos.

    The rows attend to k_ctx / v_ctx [U, Hkv, dh] (keys computed earlier, may be None) followed
    by their own keys; visible is [T, U + T].  Returns (x_out [T, d], attention output
    [T, Hq, dh], k [T, Hkv, dh], v [T, Hkv, dh]).
    """
    q, k, v = _qkv(w, shape, l, x, pos, dt, rnd)
    K = k if k_ctx is None else np.concatenate([k_ctx, k])
    V = v if v_ctx is None else np.concatenate([v_ctx, v])
    a = attend(q, K, V, visible, rnd)
    return _finish_layer(w, shape, l, x, a, dt, rnd), a, k, v


def head(w, shape, x, dt, rnd=None):
    return normed_products(x, mat(w, "gf", dt), shape.rms_eps, [mat(w, "lm_head", dt)], rnd)[0]


def forward_full(w, shape, tokens, dt=np.float64, pos0=0, return_hidden=False, rnd=None):
    """Logits [T, V] at every position of one token string (dense causal recompute)."""
    tokens = np.asarray(tokens)
    T = tokens.size
    pos = np.arange(pos0, pos0 + T)
    x = mat(w, "embed", dt)[tokens]
    causal = np.tril(np.ones((T, T), dtype=bool))
    for l in range(shape.n_layers):
        q, k, v = _qkv(w, shape, l, x, pos, dt, rnd)
        x = _finish_layer(w, shape, l, x, attend(q, k, v, causal, rnd), dt, rnd)
    return x if return_hidden else head(w, shape, x, dt, rnd)


class Incremental:
    """Token-by-token decode of one sequence with a growing K/V list per layer."""

    def __init__(self, w, shape, dt=np.float64, rnd=None):
        self.w, self.shape, self.dt, self.rnd = w, shape, dt, rnd
        self.k = [[] for _ in range(shape.n_layers)]
        self.v = [[] for _ in range(shape.n_layers)]
        self.n = 0

    def step(self, token):
        """Feed one token at position self.n; return the logits [V] after it."""
        w, shape, dt, rnd = self.w, self.shape, self.dt, self.rnd
        x = mat(w, "embed", dt)[np.asarray([token])]
        for l in range(shape.n_layers):
            q, k, v = _qkv(w, shape, l, x, [self.n], dt, rnd)
            self.k[l].append(k[0]); self.v[l].append(v[0])
            K = np.stack(self.k[l]); V = np.stack(self.v[l])
            a = attend(q, K, V, np.ones((1, K.shape[0]), dtype=bool), rnd)
            x = _finish_layer(w, shape, l, x, a, dt, rnd)
        self.n += 1
        return head(w, shape, x, dt, rnd)[0]


class SharedPrefix:
    """K/V of a cached prefix, computed once and read by all G samples of a group."""

    def __init__(self, w, shape, prefix_tokens, dt=np.float64, rnd=None):
        self.w, self.shape, self.dt, self.rnd = w, shape, dt, rnd
        prefix_tokens = np.asarray(prefix_tokens)
        self.P = P = prefix_tokens.size
        x = mat(w, "embed", dt)[prefix_tokens]
        causal = np.tril(np.ones((P, P), dtype=bool))
        self.k, self.v = [], []
        for l in range(shape.n_layers):
            q, k, v = _qkv(w, shape, l, x, np.arange(P), dt, rnd)
            self.k.append(k); self.v.append(v)
            x = _finish_layer(w, shape, l, x, attend(q, k, v, causal, rnd), dt, rnd)
        self.x_last = x[-1:].copy()                      # residual stream at the last prefix token

    def step0_logits(self):
        """Logits for suffix position 0 (shared by the whole group)."""
        return head(self.w, self.shape, self.x_last, self.dt, self.rnd)[0]

    def teacher_forced_hidden(self, suffix):
        """Residual stream after feeding suffix tokens [S'] (one sample) at positions P.."""
        w, shape, dt, P, rnd = self.w, self.shape, self.dt, self.P, self.rnd
        suffix = np.asarray(suffix)
        n = suffix.size
        x = mat(w, "embed", dt)[suffix]
        vis = np.concatenate([np.ones((n, P), dtype=bool), np.tril(np.ones((n, n), dtype=bool))], axis=1)
        for l in range(shape.n_layers):
            q, k, v = _qkv(w, shape, l, x, np.arange(P, P + n), dt, rnd)
            K = np.concatenate([self.k[l], k]); V = np.concatenate([self.v[l], v])
            x = _finish_layer(w, shape, l, x, attend(q, K, V, vis, rnd), dt, rnd)
        return x

    def teacher_forced_logits(self, suffix):
        """Logits [len(suffix), V]: row j is the distribution of o_j given prefix, o_<j."""
        suffix = np.asarray(suffix)
        xs = self.x_last
        if suffix.size > 1:
            xs = np.concatenate([xs, self.teacher_forced_hidden(suffix[:-1])])
        return head(self.w, self.shape, xs, self.dt, self.rnd)
