"""An expired device-side wait is an error the caller sees, and the context survives it.

Every wait inside the TMA / tcgen05 pipelines (mbarrier waits of the producer, MMA and epilogue or softmax
roles) is bounded.  When one runs out the CTA raises status bit 0, stops issuing work, lets the copies and
MMAs it has in flight finish while it is still resident, frees its tensor memory and returns: the launch
ends, nothing traps, the result is simply not to be trusted.  Here the limit is set so low (one clock
cycle) that the first wait that is not satisfied at once gives up; the test checks the status bit, the
error code of the calls that synchronise, and that the same context computes correctly again once the
default limit is back.  No fault, no unbounded wait is involved."""
import numpy as np
import pytest
import torch

import paper_2601_19404_b200 as rpo
import workloads
from gpu_util import DEV, make_ctx

pytestmark = pytest.mark.gpu

SHAPE = dict(n_layers=2, d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=128, d_ffn=1536, vocab=4096,
             rope_base=1e6, rms_eps=1e-6, dtype="bf16")
RPO_ERR_DEVICE_TIMEOUT = -5


def _gemm(ctx, a, w):
    out = torch.zeros((a.shape[0], w.shape[0]), dtype=torch.float32, device=DEV)
    ctx.gemm(a, w, out, impl=2)                       # the tcgen05 / TMA kernel
    return out


def test_expired_wait_is_reported_and_the_context_recovers():
    torch.manual_seed(0)
    a = (torch.randn(96, 512, device=DEV) * 0.5).to(torch.bfloat16)
    w = (torch.randn(384, 512, device=DEV) * 0.5).to(torch.bfloat16)
    want = a.float() @ w.float().T
    lens = np.array([70, 33], dtype=np.int32)
    G, S = 2, 3
    toks, off = workloads.prefix_tokens(lens, SHAPE["vocab"], seed=3)
    h_out = np.zeros((len(lens) * G, S), dtype=np.int32); h_len = np.zeros(len(lens) * G, dtype=np.int32)
    h_lp = np.zeros((len(lens) * G, S), dtype=np.float32)
    smp = rpo.Sampler(1.0, 0.9, False, -1, 5)
    with make_ctx(SHAPE, len(lens), G, int(lens.max()), S) as ctx:
        ctx.init_weights(0, 0.02)
        assert torch.allclose(_gemm(ctx, a, w), want, atol=1e-2, rtol=1e-3) and ctx.device_status() == 0
        ctx.rollout_host(toks, off, G, S, smp, h_out, h_len, h_lp)
        good = (h_out.copy(), h_lp.copy())
        try:
            ctx.set_option("wait_limit_cycles", 1)    # device-wide: restored below whatever happens
            _gemm(ctx, a, w)                          # a wait gives up; the launch still ends
            torch.cuda.synchronize()
            assert ctx.device_status(raise_on_timeout=False) & 1
            _gemm(ctx, a, w)
            with pytest.raises(rpo.RpoError) as e:    # the polling call reports it ...
                ctx.device_status()
            assert e.value.code == RPO_ERR_DEVICE_TIMEOUT
            with pytest.raises(rpo.RpoError) as e:    # ... and so does the call that synchronises anyway
                ctx.rollout_host(toks, off, G, S, smp, h_out, h_len, h_lp)
            assert e.value.code == RPO_ERR_DEVICE_TIMEOUT
        finally:
            ctx.set_option("wait_limit_cycles", 0)    # the default again
        # the same context, default limit: correct again, status clean, every KV block back in the pool
        assert ctx.device_status(raise_on_timeout=False) in (0, 1)        # (a leftover bit from the failed rollout is cleared by the read)
        assert torch.allclose(_gemm(ctx, a, w), want, atol=1e-2, rtol=1e-3)
        ctx.rollout_host(toks, off, G, S, smp, h_out, h_len, h_lp)
        assert np.array_equal(h_out, good[0]) and np.array_equal(h_lp.view(np.uint32), good[1].view(np.uint32))
        assert ctx.device_status() == 0 and ctx.counters()[1] == ctx.limits.kv_pool_blocks
