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


# --------------------------------------------------------------------------------------------
# Layer-by-layer parity through the residual-stream tap
# --------------------------------------------------------------------------------------------
def _widen(t):
    if t.dtype == np.uint16:
        t = (t.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return t.astype(np.float64)


def layer_weights_from_device(ctx, sh, l):
    """Weights of layer l as the library holds them, widened to float64 for the oracle."""
    return {f"layers.{l}.{n}": _widen(ctx.read_tensor(f"layers.{l}.{n}")) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "g1", "g2")}


class TapReader:
    """Cuts the tap buffer of rpo_debug_tap into its blocks, in the order the library wrote them."""

    def __init__(self, buf, shape_dict):
        self.buf, self.pos = buf, 0
        self.d, self.qo = shape_dict["d_model"], shape_dict["n_q_heads"] * shape_dict["head_dim"]
        self.bf16 = shape_dict["dtype"] == "bf16"
        self.L = shape_dict["n_layers"]

    def _take(self, n_floats):
        out = self.buf[self.pos:self.pos + n_floats]
        self.pos += n_floats
        return out

    def rows(self, rows):
        return self._take(rows * self.d).reshape(rows, self.d).astype(np.float64)

    def attn(self, rows):
        if not self.bf16:
            return self._take(rows * self.qo).reshape(rows, self.qo).astype(np.float64)
        raw = self._take((rows * self.qo + 1) // 2).view(np.uint16)[:rows * self.qo]
        return _widen(raw).reshape(rows, self.qo)

    def one_pass(self, rows):
        """(x [L+1][rows, d], attention outputs [L][rows, Hq*dh]) of one pass through the layer stack."""
        xs, at = [self.rows(rows)], []
        for _ in range(self.L):
            at.append(self.attn(rows))
            xs.append(self.rows(rows))
        return xs, at


def layerwise_errors(ctx, shape_dict, sh, prefix_tokens, G, S, forced):
    """One group: prefill + teacher-forced decode of G suffixes with the tap on, then every layer of the
    oracle (plain float64 definition) fed with the library's own input of that layer.

    Returns dict with, per layer, the largest deviation of the attention output and of the layer's
    output, each row's deviation measured in units of the row's rms (attention output) or of the rms of
    the row's increment x_out - x_in (layer output), for the prefix rows and for the decode rows; the
    rms deviation over all prefix rows in the same units (attn_rms, x_rms); and the final logits /
    log-prob errors against the oracle's head applied to the library's last hidden state."""
    from oracle import sampler as osampler
    P, d, L = len(prefix_tokens), shape_dict["d_model"], shape_dict["n_layers"]
    qo = shape_dict["n_q_heads"] * shape_dict["head_dim"]
    per_row = d + L * (d + (qo + 1) // 2 + 1)
    tap = torch.zeros((P + (S - 1) * G) * per_row + 1024, dtype=torch.float32, device=DEV)
    ctx.debug_tap(tap)
    off = np.array([0, P], dtype=np.int32)
    groups = ctx.prefill_prefix(dev_i32(prefix_tokens), off)
    t, l, lp, dbg = run_decode(ctx, groups, G, S, rpo.Sampler(1.0, 0.95, False, -1, 0), forced=forced, want_logits=True)
    used = ctx.debug_tap(None)
    ctx.release_groups(groups)
    rd = TapReader(tap[:used].cpu().numpy(), shape_dict)
    x_pre, a_pre = rd.one_pass(P)
    dec = [rd.one_pass(G) for _ in range(S - 1)]
    assert rd.pos == used
    # suffix rows per sample, in position order: row j of sample i is the forward of decode step j + 1
    x_suf = [np.stack([np.stack([dec[j][0][ll][i] for j in range(S - 1)]) for i in range(G)]) for ll in range(L + 1)]
    a_suf = [np.stack([np.stack([dec[j][1][ll][i] for j in range(S - 1)]) for i in range(G)]) for ll in range(L)]
    causal = np.tril(np.ones((P, P), dtype=bool))
    n = S - 1
    vis = np.concatenate([np.ones((n, P), dtype=bool), np.tril(np.ones((n, n), dtype=bool))], axis=1)
    out = dict(attn_prefill=[], x_prefill=[], attn_decode=[], x_decode=[], attn_rms=[], x_rms=[])

    def rel(got, want, scale_rows):
        return float(np.max(np.abs(got - want) / scale_rows[:, None]))

    def rel_rms(got, want, base):
        return float(np.sqrt(np.mean((got - want) ** 2)) / np.sqrt(np.mean(base ** 2)))

    def rms(a):
        return np.sqrt(np.mean(a * a, axis=-1)) + 1e-30

    for ll in range(L):
        w = layer_weights_from_device(ctx, sh, ll)
        xo, a, k_p, v_p = decoder.layer(w, sh, ll, x_pre[ll], np.arange(P), None, None, causal)
        a = a.reshape(P, qo)
        out["attn_prefill"].append(rel(a_pre[ll], a, rms(a)))
        out["x_prefill"].append(rel(x_pre[ll + 1], xo, rms(xo - x_pre[ll])))
        out["attn_rms"].append(rel_rms(a_pre[ll], a, a)); out["x_rms"].append(rel_rms(x_pre[ll + 1], xo, xo - x_pre[ll]))
        ea, ex = 0.0, 0.0
        for i in range(G):
            xo, a, _, _ = decoder.layer(w, sh, ll, x_suf[ll][i], P + np.arange(n), k_p, v_p, vis)
            a = a.reshape(n, qo)
            ea = max(ea, rel(a_suf[ll][i], a, rms(a)))
            ex = max(ex, rel(x_suf[ll + 1][i], xo, rms(xo - x_suf[ll][i])))
        out["attn_decode"].append(ea); out["x_decode"].append(ex)
        del w
    wh = {"gf": _widen(ctx.read_tensor("gf")), "lm_head": _widen(ctx.read_tensor("lm_head"))}
    last = np.concatenate([x_pre[L][-1:]] + [x_suf[L][i] for i in range(G)])        # step-0 row, then G x (S-1) rows
    ref = decoder.head(wh, sh, last, np.float64).astype(np.float32)
    ref_logits = np.stack([np.concatenate([ref[:1], ref[1 + i * n:1 + (i + 1) * n]]) for i in range(G)])    # [G, S, V]
    out["logits_err"] = float(np.max(np.abs(dbg - ref_logits)))
    ref_lp = np.array([[osampler.token_logprob(ref_logits[i, j], 1.0, int(forced[i][j])) for j in range(S)] for i in range(G)])
    out["logprob_err"] = float(np.max(np.abs(lp - ref_lp)))
    srt = np.sort(ref_logits, axis=-1)
    clear = (srt[..., -1] - srt[..., -2]) > 0.05
    out["argmax_ok"] = bool(np.all((np.argmax(dbg, -1) == np.argmax(ref_logits, -1))[clear]))
    out["clear_steps"] = int(clear.sum())
    return out
