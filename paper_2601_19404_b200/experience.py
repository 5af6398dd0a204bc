"""Host side of one RPO rollout stage around the CUDA library (Section 3, Algorithm 1).

The library computes; this module only decides *what* to roll out: it keeps the experience cache
C = {(q_k, a_k)} (Eq. 1-2), draws the truncation m ~ U{0..L} (Eq. 3) with L fixed or tied to the
shortest response of the previous sampling group (Eq. 4), builds the prefix q_k || a_k^{[0:-m]}
that rpo_prefill_prefix takes, and after the rollout replaces the cached response epsilon-greedily
(Section 3.3, Eq. 10).  Rewards come from a caller-supplied function (the paper's verifier needs
its datasets).  Token arrays are numpy int32.
"""
import numpy as np


class ExperienceCache:
    """C = {(q_k, a_k)}: one cached response per question (Eq. 1); retrieve() is Eq. 2."""

    def __init__(self):
        self._pool = {}

    def __len__(self):
        return len(self._pool)

    def __contains__(self, qid):
        return qid in self._pool

    def put(self, qid, question_tokens, answer_tokens):
        self._pool[qid] = (np.ascontiguousarray(question_tokens, dtype=np.int32), np.ascontiguousarray(answer_tokens, dtype=np.int32))

    def retrieve(self, qid):
        return self._pool[qid]


def draw_truncation(rng, L, answer_len):
    """m ~ U{0, 1, ..., L} (Eq. 3), never more than the cached answer holds."""
    return int(min(int(rng.integers(0, int(L) + 1)), int(answer_len)))


def dynamic_L(group_lens, factor=0.5):
    """L tied to the shortest response of a sampling group (Eq. 4; the experiments use 0.5 * l)."""
    return int(factor * int(np.min(group_lens)))


def build_prefix(question_tokens, answer_tokens, m):
    """q_k || a_k^{[0:-m]}: the last m tokens of the cached answer are dropped; m = 0 keeps all of it."""
    a = np.asarray(answer_tokens, dtype=np.int32)
    keep = a.size - int(m)
    return np.concatenate([np.asarray(question_tokens, dtype=np.int32), a[:max(keep, 0)]])


def epsilon_greedy_choice(rng, rewards, eps):
    """Index of the response that replaces the cached one (Eq. 10): with probability eps (u <= eps) the
    highest-reward response (lowest index among ties), otherwise one of the others, uniformly."""
    rewards = np.asarray(rewards)
    best = int(np.argmax(rewards))
    if rewards.size == 1 or rng.random() <= eps:
        return best
    others = [i for i in range(rewards.size) if i != best]
    return int(others[int(rng.integers(0, len(others)))])


class RolloutStage:
    """retrieve -> truncate -> prefill once per group -> G suffixes -> log-probs -> rewards -> objective
    forward -> cache update, for a batch of questions.  `ctx` is a paper_2601_19404_b200.Context."""

    def __init__(self, ctx, cache, G, max_new, sampler, reward_fn, L=300, dynamic_factor=None, eps=0.1, seed=0, objective_cfg=None):
        self.ctx, self.cache, self.G, self.max_new, self.sampler, self.reward_fn = ctx, cache, int(G), int(max_new), sampler, reward_fn
        self.L, self.dynamic_factor, self.eps = int(L), dynamic_factor, float(eps)
        self.rng = np.random.Generator(np.random.PCG64([int(seed), 707]))
        self.objective_cfg = objective_cfg
        self._last_min_len = {}

    def run(self, qids):
        import torch
        from . import binding
        ctx, G, S = self.ctx, self.G, self.max_new
        dev = torch.device("cuda", torch.cuda.current_device())
        prefixes, kept, ms = [], [], []
        for q in qids:
            qt, at = self.cache.retrieve(q)
            L = self.L if self.dynamic_factor is None or q not in self._last_min_len else dynamic_L([self._last_min_len[q]], self.dynamic_factor)
            m = draw_truncation(self.rng, L, at.size)
            prefixes.append(build_prefix(qt, at, m)); kept.append(at.size - m); ms.append(m)
        off = np.zeros(len(qids) + 1, dtype=np.int32); off[1:] = np.cumsum([p.size for p in prefixes])
        toks = np.concatenate(prefixes).astype(np.int32)
        B = len(qids) * G
        d_out = torch.zeros((B, S), dtype=torch.int32, device=dev); d_lens = torch.zeros(B, dtype=torch.int32, device=dev)
        d_lp = torch.zeros((B, S), dtype=torch.float32, device=dev); d_pol = torch.zeros((B, S), dtype=torch.float32, device=dev)
        groups = ctx.prefill_prefix(torch.from_numpy(toks).to(dev), off, np.arange(len(qids), dtype=np.int32))
        ctx.decode_suffix(groups, G, S, self.sampler, d_out, d_lens, d_lp)
        ctx.token_logprobs(groups, G, S, d_out, d_lens, d_pol, inv_temperature=1.0 / self.sampler.temperature)
        ctx.release_groups(groups)
        torch.cuda.synchronize()
        out, lens = d_out.cpu().numpy(), d_lens.cpu().numpy()
        # responses o = a^{[0:-m]} || generated suffix; reward and full response length per sample
        responses, raw, resp_lens = [], np.zeros(B, dtype=np.float32), np.zeros(B, dtype=np.int32)
        for k, q in enumerate(qids):
            qt, at = self.cache.retrieve(q)
            for i in range(G):
                b = k * G + i
                o = np.concatenate([at[:kept[k]], out[b, :lens[b]]]).astype(np.int32)
                responses.append(o); raw[b] = float(self.reward_fn(q, qt, o)); resp_lens[b] = o.size
        result = dict(tokens=out, lens=lens, logprobs=d_lp.cpu().numpy(), policy_logprobs=d_pol.cpu().numpy(), truncations=ms,
                      raw_rewards=raw, resp_lens=resp_lens)
        if self.objective_cfg is not None:
            R = torch.zeros(B, device=dev); A = torch.zeros(B, device=dev); gobj = torch.zeros(len(qids), device=dev); J = torch.zeros(1, device=dev)
            ctx.policy_objective(len(qids), G, S, d_pol, d_lp, d_lens, torch.from_numpy(raw).to(dev), self.objective_cfg, R, A, gobj, J,
                                 d_resp_lens=torch.from_numpy(resp_lens).to(dev))
            torch.cuda.synchronize()
            result.update(rewards=R.cpu().numpy(), advantages=A.cpu().numpy(), group_objective=gobj.cpu().numpy(), objective=float(J.item()))
        # cache update (Eq. 10) on the shaped rewards when available, else the raw ones
        score = result.get("rewards", raw)
        chosen = []
        for k, q in enumerate(qids):
            pick = epsilon_greedy_choice(self.rng, score[k * G:(k + 1) * G], self.eps)
            qt, _ = self.cache.retrieve(q)
            self.cache.put(q, qt, responses[k * G + pick])
            self._last_min_len[q] = int(resp_lens[k * G:(k + 1) * G].min())
            chosen.append(pick)
        result["chosen"] = chosen
        return result
