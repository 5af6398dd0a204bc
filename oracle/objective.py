"""Forward value of the RPO / GRPO objective of one rollout batch (test infrastructure).

Plain float64 restatement of Section 3.2 (Eq. 5-7) and Section 3.4 (Eq. 11):

  length-aware reward (Eq. 11)   R_i = clip( r_i / (1 + exp(-alpha (l_ref - len_i))), m, M ),
                                 l_ref = mean of len over the sampling group
  advantage (Eq. 7)              A_i = (R_i - mu_R) / sigma_R over the group
  ratio (Eq. 7)                  r_ij = pi_theta(o_ij | q, o_i<j) / pi_theta_old(o_ij | q, o_i<j)
  token loss (Eq. 6)             l_ij = min( r_ij A_i, clip(r_ij, 1 - eps, 1 + eps) A_i )
  objective (Eq. 5)              J = mean over groups of [ 1/G sum_i 1/|o_i| sum_j l_ij ] - beta * KL

Readings where the paper is silent: sigma_R is the population standard deviation and A_i = 0 for a
group whose rewards are all equal; the sums over j run over the tokens generated in this rollout
(|o_i| = their number); len_i of Eq. 11 is the response length handed in by the caller (by default
the same number); the KL term is the per-token estimator of GRPO, which the paper builds on,
k3 = pi_ref/pi_theta - log(pi_ref/pi_theta) - 1, averaged with the same 1/|o_i| and 1/G weights.
"""
import numpy as np


def length_aware_rewards(raw, resp_lens, G, alpha, r_min, r_max):
    raw = np.asarray(raw, dtype=np.float64).reshape(-1, G)
    ln = np.asarray(resp_lens, dtype=np.float64).reshape(-1, G)
    l_ref = ln.mean(axis=1, keepdims=True)
    shaped = raw / (1.0 + np.exp(-alpha * (l_ref - ln)))
    return np.clip(shaped, r_min, r_max).reshape(-1)


def group_advantages(rewards, G):
    R = np.asarray(rewards, dtype=np.float64).reshape(-1, G)
    mu = R.mean(axis=1, keepdims=True)
    sd = np.sqrt(((R - mu) ** 2).mean(axis=1, keepdims=True))
    with np.errstate(divide="ignore", invalid="ignore"):
        A = np.where(sd > 0, (R - mu) / sd, 0.0)
    return A.reshape(-1)


def objective(logp_new, logp_old, lens, raw_rewards, G, clip_eps=0.2, beta=0.0, logp_ref=None, length_shaping=True,
              alpha=0.01, r_min=0.5, r_max=1.0, resp_lens=None):
    """Returns dict(rewards [B], advantages [B], token_loss [B,S], group_objective [n_groups], objective)."""
    logp_new = np.asarray(logp_new, dtype=np.float64); logp_old = np.asarray(logp_old, dtype=np.float64)
    B, S = logp_new.shape
    lens = np.asarray(lens)
    resp = lens if resp_lens is None else np.asarray(resp_lens)
    R = length_aware_rewards(raw_rewards, resp, G, alpha, r_min, r_max) if length_shaping else np.asarray(raw_rewards, dtype=np.float64)
    A = group_advantages(R, G)
    tok = np.zeros((B, S))
    per_seq = np.zeros(B)
    for i in range(B):
        n = int(lens[i])
        if n == 0:
            continue
        ratio = np.exp(logp_new[i, :n] - logp_old[i, :n])
        l = np.minimum(ratio * A[i], np.clip(ratio, 1.0 - clip_eps, 1.0 + clip_eps) * A[i])
        if logp_ref is not None and beta != 0.0:
            d = np.asarray(logp_ref, dtype=np.float64)[i, :n] - logp_new[i, :n]
            l = l - beta * (np.exp(d) - d - 1.0)
        tok[i, :n] = l
        per_seq[i] = l.sum() / n
    grp = per_seq.reshape(-1, G).mean(axis=1)
    return dict(rewards=R, advantages=A, token_loss=tok, group_objective=grp, objective=float(grp.mean()))
