"""Sampler of the rollout policy pi_theta(. | q_k, prefix, o_<j) (Eq. 3), exact integers.

The paper fixes only the temperature (Section 4).  Reading used by this project:
temperature T, softmax, nucleus (top-p) with a ties-inclusive probability threshold,
inverse CDF in ascending token id.  Because a floating-point sum order would decide
token ids differently on different machines, probabilities are *quantised*:

    z_i = logit_i / T               (float32 division)
    e_i = exp_nonpos(z_i - max z)   (reproducible float32 exp, exactly 0 below -24)
    w_i = floor(e_i * 2^30)         (integer weight, 0 .. 2^30)

and everything after that is integer arithmetic, hence independent of summation order:

    total  = sum_i w_i
    target = (total * floor(top_p * 2^24)) >> 24
    S(t)   = sum_{w_i >= t} w_i
    tau    = the largest weight value t occurring in w with S(t) >= target
    nucleus = { i : w_i >= tau },  mass = S(tau)
    r      = (mass * u24) >> 24     with u24 the 24-bit Philox draw, so 0 <= r < mass
    token  = the first nucleus member, in ascending id, whose running weight sum exceeds r

Greedy mode returns the lowest id among maximal logits.  The reported log-probability
is over the full vocabulary (no nucleus renormalisation): z_tok - logsumexp(z).
"""
import numpy as np
from . import exactmath as em

F = np.float32
W_SCALE_LOG2 = 30


def quantised_weights(logits, temperature):
    """Integer weights w_i (uint64) for one row of float32 logits."""
    z = (np.asarray(logits, dtype=F) / F(temperature)).astype(F)
    zmax = z.max()
    e = em.exp_nonpos((z - zmax).astype(F))
    return (e * F(2.0 ** W_SCALE_LOG2)).astype(F).astype(np.uint64)


def top_p_fixed(top_p):
    return int(np.floor(F(top_p) * F(2.0 ** 24)))


def nucleus_threshold(w, top_p):
    """(tau, mass) of the ties-inclusive nucleus for integer weights w."""
    total = int(w.sum(dtype=np.uint64))
    target = (total * top_p_fixed(top_p)) >> 24
    vals, inv = np.unique(w, return_inverse=True)          # ascending distinct weights
    mass_per_val = np.zeros(vals.size, dtype=np.uint64)
    np.add.at(mass_per_val, inv, w)
    s_from_top = np.cumsum(mass_per_val[::-1], dtype=np.uint64)[::-1]   # S(vals[k])
    ok = np.nonzero(s_from_top >= np.uint64(target))[0]                # always contains 0
    k = ok.max()
    return int(vals[k]), int(s_from_top[k])


def sample_token(logits, temperature, top_p, u24):
    w = quantised_weights(logits, temperature)
    tau, mass = nucleus_threshold(w, top_p)
    r = (mass * int(u24)) >> 24
    kept = np.where(w >= np.uint64(tau), w, np.uint64(0))
    run = np.cumsum(kept, dtype=np.uint64)
    return int(np.argmax(run > np.uint64(r)))              # first index where the running sum exceeds r


def greedy_token(logits):
    return int(np.argmax(np.asarray(logits)))               # numpy argmax = first (lowest id) maximum


def log_softmax_row(logits, temperature=1.0):
    z = np.asarray(logits, dtype=np.float64) / float(temperature)
    m = z.max()
    return z - (m + np.log(np.exp(z - m).sum()))


def token_logprob(logits, temperature, token):
    return float(log_softmax_row(logits, temperature)[token])
