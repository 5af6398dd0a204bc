"""Continuous batching of the cache initialisation (host logic) against a deterministic stand-in
for the generator: tokens are a function of (group id, position), every request stops at its own
length."""
import os
import sys

import numpy as np
import pytest

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from paper_2601_19404_b200 import cache_init

EOS = 7


def make_engine(stop_after, log=None):
    """Request r emits EOS as its stop_after[r]-th token; other tokens depend on (r, wave, position)."""
    def engine(prefixes, ids, max_new):
        n = len(prefixes)
        toks = np.full((n, max_new), EOS, dtype=np.int32)
        lens = np.zeros(n, dtype=np.int32)
        for k in range(n):
            r, wave = divmod(int(ids[k]), cache_init.MAX_WAVES)
            done_before = wave * max_new
            # the prefix must be the prompt followed by everything generated so far
            assert prefixes[k].size == 3 + r + done_before
            for j in range(max_new):
                pos = done_before + j
                if pos + 1 == stop_after[r]:
                    toks[k, j] = EOS; lens[k] = j + 1
                    break
                toks[k, j] = 100 + (r * 31 + wave * 17 + j * 3) % 50
                lens[k] = j + 1
        if log is not None:
            log.append(sorted(int(i) // cache_init.MAX_WAVES for i in ids))
        return toks, lens
    return engine


def prompts(n):
    return [np.arange(3 + r, dtype=np.int32) for r in range(n)]


def test_responses_do_not_depend_on_the_batch_size():
    stop = [5, 40, 13, 64, 1, 29, 8, 200]            # request 7 never stops within max_len
    ref, _ = cache_init.schedule(prompts(8), make_engine(stop), 1, 8, 96, EOS)
    for r in range(7):
        assert ref[r].size == stop[r] and ref[r][-1] == EOS and np.all(ref[r][:-1] != EOS)
    assert ref[7].size == 96 and EOS not in ref[7]   # cut at max_len, no EOS
    for mb in (2, 3, 8, 50):
        got, st = cache_init.schedule(prompts(8), make_engine(stop), mb, 8, 96, EOS)
        assert all(np.array_equal(a, b) for a, b in zip(got, ref))
        assert st["useful_tokens"] == sum(x.size for x in ref) <= st["slot_tokens"]


def test_finished_sequences_hand_their_slots_to_waiting_requests():
    stop = [4, 60, 4, 4, 4, 60]
    log = []
    _, st = cache_init.schedule(prompts(6), make_engine(stop, log), 2, 8, 64, EOS)
    assert log[0] == [0, 1]                          # first wave: the first two requests
    assert log[1] == [1, 2]                          # request 0 stopped, request 2 took its slot
    assert log[2] == [1, 3] and log[3] == [1, 4] and log[4] == [1, 5]
    assert all(len(b) <= 2 for b in log)
    # a static batch of 2 would need ceil(60/8) waves per pair = 24; continuous batching needs 12
    assert st["waves"] == 12
    with pytest.raises(ValueError):
        cache_init.schedule(prompts(1), make_engine([3]), 0, 8, 64, EOS)


def test_no_eos_configured_runs_every_request_to_max_len():
    got, st = cache_init.schedule(prompts(3), make_engine([1000, 1000, 1000]), 2, 5, 12, -1)
    assert all(g.size == 12 for g in got) and st["useful_tokens"] == 36


class ToySession:
    """Stand-in for a generator that keeps its sequences' state: request r's token at absolute position p is a
    function of (r, p) alone; it checks that requests are admitted once, advanced in order and retired once."""

    def __init__(self, stop_after, log=None):
        self.stop, self.pos, self.log, self.retired, self.prefills = stop_after, {}, log, [], 0

    def admit(self, requests, prompts_):
        for r, p in zip(requests, prompts_):
            assert r not in self.pos and r not in self.retired and p.size == 3 + r
            self.pos[r] = 0
            self.prefills += 1

    def wave(self, requests, max_new):
        assert requests == sorted(requests) and all(r in self.pos for r in requests)
        toks = np.full((len(requests), max_new), EOS, dtype=np.int32)
        lens = np.zeros(len(requests), dtype=np.int32)
        for k, r in enumerate(requests):
            for j in range(max_new):
                p = self.pos[r] + j
                if p + 1 == self.stop[r]:
                    toks[k, j] = EOS; lens[k] = j + 1
                    break
                toks[k, j] = 100 + (r * 31 + p * 3) % 50
                lens[k] = j + 1
            self.pos[r] += max_new
        if self.log is not None:
            self.log.append(list(requests))
        return toks, lens

    def retire(self, requests):
        for r in requests:
            del self.pos[r]
            self.retired.append(r)


def test_resumable_schedule_prefills_once_and_is_independent_of_batch_and_wave_size():
    stop = [5, 40, 13, 64, 1, 29, 8, 200]
    want = []
    for r in range(8):                                # the response of request r, written out directly
        n = min(stop[r], 96)
        t = np.array([100 + (r * 31 + p * 3) % 50 for p in range(n)], dtype=np.int32)
        if stop[r] <= 96:
            t[-1] = EOS
        want.append(t)
    for mb, wave in ((1, 8), (2, 8), (3, 5), (8, 96), (50, 7)):
        s = ToySession(stop)
        got, st = cache_init.schedule_resumable(prompts(8), s, mb, wave, 96, EOS)
        assert all(np.array_equal(a, b) for a, b in zip(got, want)), (mb, wave)
        assert s.prefills == 8 and sorted(s.retired) == list(range(8)) and not s.pos
        assert st["useful_tokens"] == sum(x.size for x in want) <= st["slot_tokens"]


def test_resumable_schedule_hands_slots_over_like_the_stateless_one():
    stop = [4, 60, 4, 4, 4, 60]
    log = []
    _, st = cache_init.schedule_resumable(prompts(6), ToySession(stop, log), 2, 8, 64, EOS)
    assert log[:5] == [[0, 1], [1, 2], [1, 3], [1, 4], [1, 5]] and st["waves"] == 12
    with pytest.raises(ValueError):
        cache_init.schedule_resumable(prompts(1), ToySession([3]), 2, 0, 64, EOS)
