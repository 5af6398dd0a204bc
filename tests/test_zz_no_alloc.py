"""rpo_sample_rows_noalloc: the sampler for hosts that cannot allocate device memory.

A serving process that has given the whole GPU to its own pool, or a plug-in that only receives
buffers and a stream, cannot let this library allocate.  The variant tested here keeps its
per-token scratch in a fixed array inside the library and takes no context.  It must return
exactly what rpo_sample_rows returns, call after call, although every call reuses the same
scratch with the previous call's contents still in it.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import paper_2601_19404_b200 as rpo
import workloads
from oracle import philox, sampler as osampler
from gpu_util import DEV, make_ctx

pytestmark = pytest.mark.gpu

NOALLOC_MAX_WORDS = 4 << 20


def _both(ctx, logits, smp, seqs, step, stream):
    n = logits.shape[0]
    d_logits = torch.from_numpy(logits).to(DEV); d_seq = torch.from_numpy(seqs).to(DEV)
    want_t = torch.zeros(n, dtype=torch.int32, device=DEV); want_lp = torch.zeros(n, dtype=torch.float32, device=DEV)
    got_t = torch.full((n,), -5, dtype=torch.int32, device=DEV); got_lp = torch.full((n,), 9.0, dtype=torch.float32, device=DEV)
    torch.cuda.synchronize()
    ctx.sample_rows(d_logits, smp, d_seq, step, want_t, want_lp)
    rpo.sample_rows_noalloc(d_logits, smp, d_seq, step, got_t, got_lp, stream=stream)
    torch.cuda.synchronize()
    return want_t.cpu().numpy(), want_lp.cpu().numpy(), got_t.cpu().numpy(), got_lp.cpu().numpy()


def test_noalloc_sampler_equals_the_allocating_entry_point_on_consecutive_calls():
    tiny = workloads.SHAPES["tiny"]
    stream = torch.cuda.Stream()
    with make_ctx(tiny, 1, 1, 32, 4) as ctx:
        # two calls in a row on the same scratch: a wide vocabulary first, then a narrower one whose
        # rows land on words the first call left behind; then a greedy call
        calls = [(5, 151936, 0.78, False, 1.0, 0.95, 3), (7, 5000, 2.0, True, 0.7, 0.9, 4), (3, 1024, 1.0, False, 1.3, 0.5, 0)]
        for ci, (n, V, sigma, ties, T, top_p, step) in enumerate(calls):
            logits = workloads.logits_rows(n, V, sigma, seed=40 + ci, bf16_like=ties)
            seqs = np.arange(n, dtype=np.int64) * 3 + 11
            smp = rpo.Sampler(T, top_p, False, -1, seed=7 + ci)
            want_t, want_lp, got_t, got_lp = _both(ctx, logits, smp, seqs, step, stream)
            assert np.array_equal(got_t, want_t), ci                      # token ids: bit-exact
            for r in range(n):                                            # ... and the oracle's decision on these logits
                u24 = int(philox.sampler_u24(7 + ci, int(seqs[r]), step))
                assert got_t[r] == osampler.sample_token(logits[r], T, top_p, u24), (ci, r)
            assert np.max(np.abs(got_lp - want_lp)) <= 1e-4, ci           # the tolerance of the sampler parity test
        logits = workloads.logits_rows(4, 4096, 1.0, seed=50)
        want_t, _, got_t, _ = _both(ctx, logits, rpo.Sampler(1.0, 1.0, True, -1, 0), np.arange(4, dtype=np.int64), 0, None)
        assert np.array_equal(got_t, want_t)
        assert ctx.device_status() == 0


def test_noalloc_sampler_rejects_requests_beyond_its_built_in_scratch():
    V = 151936
    n = NOALLOC_MAX_WORDS // V + 1
    d_logits = torch.zeros((n, V), dtype=torch.float32, device=DEV)
    d_seq = torch.zeros(n, dtype=torch.int64, device=DEV)
    toks = torch.full((n,), -5, dtype=torch.int32, device=DEV)
    with pytest.raises(rpo.RpoError) as e:
        rpo.sample_rows_noalloc(d_logits, rpo.Sampler(1.0, 0.9, False, -1, 0), d_seq, 0, toks)
    assert e.value.code == -7                                             # RPO_ERR_LIMIT
    torch.cuda.synchronize()
    assert int(toks[0]) == -5                                             # nothing was launched
