"""Initialisation of the experience cache: one full-path response per question (Section 3.1,
Eq. 1; the paper generates them once, before training, spread over its GPUs), with continuous
batching on top of the rollout library.

Full responses end at very different lengths, so a fixed batch would idle on its longest member.
Here generation proceeds in *waves* of `wave_tokens` tokens: after every wave the sequences that
emitted EOS (or reached `max_len`) leave the batch and waiting questions take their slots.  With
`schedule`, a sequence that continues is re-prefilled from its prompt plus what it has generated so
far, which keeps the library's interface unchanged: every wave is `rpo_prefill_prefix` +
`rpo_decode_suffix` with one sample per group.  That re-reading is not free: with 512-token
prompts, batches of 32 and waves of 32 tokens on the 1.5B-class decoder it takes 41 % of the time
(8.5 k against 14.4 k tokens/s for `schedule_resumable` below, measured by bench.py).

Determinism: wave w of request r samples from the random stream of group id r * MAX_WAVES + w,
so a response depends only on (seed, request index, wave size), never on which other requests
shared its batches.

`schedule_resumable` is the same scheduler on top of `rpo_decode_wave`, which keeps a sequence's
private K/V and its last residual row between waves: a request is prefilled once, when it is
admitted, and every wave only decodes.  There the whole response of request r comes from the one
stream of group id r * MAX_WAVES, draw number = absolute position, i.e. it equals a single
`rpo_decode_suffix` call of `max_len` tokens and does not depend on the wave size either.
"""
import collections

import numpy as np

MAX_WAVES = 1 << 12


def schedule(prompts, engine, max_batch, wave_tokens, max_len, eos_id):
    """Continuous batching over `engine`.

    prompts: list of int32 arrays (request r = prompts[r]).
    engine(prefixes, group_ids, max_new) -> (tokens [n, max_new] int32, lens [n] int32): generates
        up to max_new tokens after each prefix; lens counts tokens up to and including EOS.
    Returns (responses, stats): responses[r] = generated tokens of request r (ends with eos_id if the
    model stopped by itself), stats = dict(waves=..., slot_tokens=..., useful_tokens=...)."""
    if max_batch <= 0 or wave_tokens <= 0 or max_len <= 0:
        raise ValueError("max_batch, wave_tokens and max_len must be positive")
    if -(-max_len // wave_tokens) > MAX_WAVES:
        raise ValueError("too many waves per request")
    waiting = collections.deque(range(len(prompts)))
    active = []                                              # request indices, in admission order
    gen = [np.zeros(0, dtype=np.int32) for _ in prompts]
    wave_of = [0] * len(prompts)
    stats = dict(waves=0, slot_tokens=0, useful_tokens=0)
    while waiting or active:
        while waiting and len(active) < max_batch:
            active.append(waiting.popleft())
        order = sorted(active)                               # batch layout independent of admission history
        prefixes = [np.concatenate([np.asarray(prompts[r], dtype=np.int32), gen[r]]) for r in order]
        ids = np.asarray([r * MAX_WAVES + wave_of[r] for r in order], dtype=np.int32)
        toks, lens = engine(prefixes, ids, wave_tokens)
        stats["waves"] += 1
        stats["slot_tokens"] += len(order) * wave_tokens
        still = []
        for k, r in enumerate(order):
            room = max_len - gen[r].size
            n = int(min(int(lens[k]), room))
            new = np.asarray(toks[k][:n], dtype=np.int32)
            gen[r] = np.concatenate([gen[r], new])
            wave_of[r] += 1
            stats["useful_tokens"] += n
            stopped = n > 0 and eos_id >= 0 and new[-1] == eos_id
            if not stopped and gen[r].size < max_len:
                still.append(r)
        keep = set(still)
        active = [r for r in active if r in keep]
    return gen, stats


def schedule_resumable(prompts, session, max_batch, wave_tokens, max_len, eos_id):
    """Continuous batching over a generator that keeps its sequences' state between waves.

    session.admit(requests, prompts) starts the given requests (a list of request indices and their prompts),
    session.wave(requests, max_new) -> (tokens [n, max_new], lens [n]) generates the next tokens of each,
    session.retire(requests) drops them.  Same return value as schedule()."""
    if max_batch <= 0 or wave_tokens <= 0 or max_len <= 0:
        raise ValueError("max_batch, wave_tokens and max_len must be positive")
    waiting = collections.deque(range(len(prompts)))
    active = []
    gen = [np.zeros(0, dtype=np.int32) for _ in prompts]
    stats = dict(waves=0, slot_tokens=0, useful_tokens=0)
    while waiting or active:
        fresh = []
        while waiting and len(active) + len(fresh) < max_batch:
            fresh.append(waiting.popleft())
        if fresh:
            session.admit(fresh, [np.asarray(prompts[r], dtype=np.int32) for r in fresh])
            active.extend(fresh)
        order = sorted(active)
        n_new = min(wave_tokens, max(max_len - gen[r].size for r in order))
        toks, lens = session.wave(order, n_new)
        stats["waves"] += 1
        stats["slot_tokens"] += len(order) * n_new
        gone = []
        for k, r in enumerate(order):
            n = int(min(int(lens[k]), max_len - gen[r].size))
            new = np.asarray(toks[k][:n], dtype=np.int32)
            gen[r] = np.concatenate([gen[r], new])
            stats["useful_tokens"] += n
            stopped = n > 0 and eos_id >= 0 and new[-1] == eos_id
            if stopped or gen[r].size >= max_len:
                gone.append(r)
        if gone:
            session.retire(gone)
            active = [r for r in active if r not in set(gone)]
    return gen, stats


class LibrarySession:
    """session for schedule_resumable(): one group per request (G = 1) through ctx (a Context); a request is
    prefilled when admitted and decoded wave by wave with rpo_decode_wave."""

    def __init__(self, ctx, sampler, max_len):
        import torch
        self.torch, self.ctx, self.sampler, self.max_len = torch, ctx, sampler, int(max_len)
        self.dev = torch.device("cuda", torch.cuda.current_device())
        self.groups = {}

    def admit(self, requests, prompts):
        off = np.zeros(len(prompts) + 1, dtype=np.int32)
        off[1:] = np.cumsum([p.size for p in prompts])
        ids = np.asarray([r * MAX_WAVES for r in requests], dtype=np.int32)
        toks = self.torch.from_numpy(np.concatenate(prompts).astype(np.int32)).to(self.dev)
        handles = self.ctx.prefill_prefix(toks, off, ids)
        for k, r in enumerate(requests):
            self.groups[r] = handles[k]

    def _handles(self, requests):
        arr = (type(self.groups[requests[0]]) * len(requests))()
        for k, r in enumerate(requests):
            arr[k] = self.groups[r]
        return arr

    def wave(self, requests, max_new):
        n = len(requests)
        d_out = self.torch.zeros((n, max_new), dtype=self.torch.int32, device=self.dev)
        d_len = self.torch.zeros(n, dtype=self.torch.int32, device=self.dev)
        self.ctx.decode_wave(self._handles(requests), 1, max_new, self.max_len, self.sampler, d_out, d_len)
        self.torch.cuda.synchronize()
        return d_out.cpu().numpy(), d_len.cpu().numpy()

    def retire(self, requests):
        self.ctx.release_groups(self._handles(requests))
        for r in requests:
            del self.groups[r]


def library_engine(ctx, sampler):
    """engine for schedule(): one group per sequence (G = 1) through ctx (a Context)."""
    import torch
    dev = torch.device("cuda", torch.cuda.current_device())

    def engine(prefixes, group_ids, max_new):
        n = len(prefixes)
        off = np.zeros(n + 1, dtype=np.int32)
        off[1:] = np.cumsum([p.size for p in prefixes])
        toks = np.concatenate(prefixes).astype(np.int32)
        d_out = torch.zeros((n, max_new), dtype=torch.int32, device=dev)
        d_len = torch.zeros(n, dtype=torch.int32, device=dev)
        groups = ctx.prefill_prefix(torch.from_numpy(toks).to(dev), off, group_ids)
        ctx.decode_suffix(groups, 1, max_new, sampler, d_out, d_len)
        ctx.release_groups(groups)
        torch.cuda.synchronize()
        return d_out.cpu().numpy(), d_len.cpu().numpy()

    return engine


def initialise_cache(cache, ctx, sampler, questions, max_batch, wave_tokens, max_len, resume=False):
    """Fills `cache` (an ExperienceCache) with one sampled response per question.
    questions: dict qid -> prompt tokens.  resume: decode in kept-state waves (schedule_resumable) instead of
    prefilling prompt + generated tokens again at every wave.  Returns the scheduler's statistics."""
    qids = sorted(questions)
    if resume:
        responses, stats = schedule_resumable([questions[q] for q in qids], LibrarySession(ctx, sampler, max_len), max_batch,
                                              wave_tokens, max_len, sampler.eos_id)
    else:
        responses, stats = schedule([questions[q] for q in qids], library_engine(ctx, sampler), max_batch, wave_tokens,
                                    max_len, sampler.eos_id)
    for q, a in zip(qids, responses):
        cache.put(q, questions[q], a)
    return stats
