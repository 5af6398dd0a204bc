"""Suffix rollout of one sampling group and its token log-probabilities.

Rollout (Eq. 3, Algorithm 1 inner loop): for a cached prefix (question plus truncated
cached answer, already concatenated) generate G continuations; sample i of group g is
sequence number g*G + i for the random stream.  A sequence ends after emitting the
EOS id: that token and its log-probability are recorded, later slots hold the EOS id
and log-probability 0, and the length counts tokens up to and including EOS.

Token log-probabilities (Eq. 7): log pi(o_j | q, o_<j) with the full-vocabulary
normalisation, teacher-forced on given suffix tokens.
"""
from dataclasses import dataclass
import numpy as np
from . import decoder, sampler, philox


@dataclass(frozen=True)
class SamplerCfg:
    temperature: float = 1.0
    top_p: float = 1.0
    greedy: bool = False
    seed: int = 0
    eos_id: int = -1


def rollout_group(w, shape, prefix_tokens, G, max_new, cfg, group_id=0, dt=np.float64,
                  forced_tokens=None, want_logits=False, rnd=None):
    """Generate (or teacher-force) G suffixes over one shared prefix.

    Returns dict(tokens [G,max_new] int32, lens [G] int32, logprobs [G,max_new] float64,
    logits [G,max_new,V] float32 if want_logits).  Logits are rounded to float32 before
    the sampler, which is the precision the sampler is defined in.  `rnd` (a
    `decoder.Rounding`) switches the decoder's optional storage rounding on.
    """
    sp = decoder.SharedPrefix(w, shape, prefix_tokens, dt, rnd)
    tokens = np.zeros((G, max_new), dtype=np.int32)
    logprobs = np.zeros((G, max_new), dtype=np.float64)
    lens = np.zeros(G, dtype=np.int32)
    all_logits = np.zeros((G, max_new, shape.vocab), dtype=np.float32) if want_logits else None
    step0 = sp.step0_logits().astype(np.float32)
    for i in range(G):
        seq = group_id * G + i
        inc_k = [list(k) for k in sp.k]      # private copy of the prefix K/V for this sample
        inc_v = [list(v) for v in sp.v]
        inc = decoder.Incremental(w, shape, dt, rnd)
        inc.k, inc.v, inc.n = inc_k, inc_v, sp.P
        logits = step0
        done = False
        for j in range(max_new):
            if done:
                tokens[i, j] = cfg.eos_id
                continue
            if want_logits:
                all_logits[i, j] = logits
            if forced_tokens is not None:
                tok = int(forced_tokens[i][j])
            elif cfg.greedy:
                tok = sampler.greedy_token(logits)
            else:
                u24 = int(philox.sampler_u24(cfg.seed, seq, j))
                tok = sampler.sample_token(logits, cfg.temperature, cfg.top_p, u24)
            tokens[i, j] = tok
            logprobs[i, j] = sampler.token_logprob(logits, cfg.temperature, tok)
            lens[i] = j + 1
            if tok == cfg.eos_id:
                done = True
            elif j + 1 < max_new:
                logits = inc.step(tok).astype(np.float32)
    out = dict(tokens=tokens, lens=lens, logprobs=logprobs)
    if want_logits:
        out["logits"] = all_logits
    return out


def token_logprobs(w, shape, prefix_tokens, suffix_tokens, lens, inv_temperature=1.0, dt=np.float64,
                   want_logits=False, rnd=None):
    """log pi(o_j | prefix, o_<j) for j < lens[i]; zeros beyond. suffix_tokens [G, S]."""
    sp = decoder.SharedPrefix(w, shape, prefix_tokens, dt, rnd)
    suffix_tokens = np.asarray(suffix_tokens)
    G, S = suffix_tokens.shape
    out = np.zeros((G, S), dtype=np.float64)
    logits_out = []
    for i in range(G):
        n = int(lens[i])
        if n == 0:
            logits_out.append(None)
            continue
        logits = sp.teacher_forced_logits(suffix_tokens[i, :n]).astype(np.float32)
        logits_out.append(logits)
        for j in range(n):
            out[i, j] = sampler.token_logprob(logits[j], 1.0 / inv_temperature, suffix_tokens[i, j])
    return (out, logits_out) if want_logits else out
