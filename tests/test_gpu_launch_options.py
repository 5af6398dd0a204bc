"""How the kernels are launched must not change what they compute: CUDA graph per decode step on / off and
programmatic dependent launch off / on (in its default form: many-row passes and the captured step graphs)
give bit-identical tokens, lengths and log-probs on a sampled rollout."""
import numpy as np
import pytest
import torch

import paper_2601_19404_b200 as rpo
import workloads
from gpu_util import DEV, make_ctx, dev_i32, run_decode

pytestmark = pytest.mark.gpu

SHAPE = dict(n_layers=4, d_model=512, n_q_heads=8, n_kv_heads=2, head_dim=128, d_ffn=1536, vocab=256,
             rope_base=1e6, rms_eps=1e-6, dtype="bf16")


def test_graphs_and_programmatic_launch_do_not_change_results():
    lens = np.array([300, 37, 90], dtype=np.int32)
    G, S, EOS = 4, 40, 5
    toks, off = workloads.prefix_tokens(lens, SHAPE["vocab"], seed=4)
    results = []
    for use_graph, use_pdl in ((1, 1), (0, 1), (1, 0), (0, 0)):
        with make_ctx(SHAPE, len(lens), G, int(lens.max()), S) as ctx:
            ctx.set_option("use_graph", use_graph)
            ctx.set_option("use_pdl", use_pdl)
            ctx.init_weights(0, 0.02)
            groups = ctx.prefill_prefix(dev_i32(toks), off)
            t, l, lp, _ = run_decode(ctx, groups, G, S, rpo.Sampler(1.0, 0.95, False, EOS, 9))
            pol = torch.zeros((len(lens) * G, S), dtype=torch.float32, device=DEV)
            ctx.token_logprobs(groups, G, S, dev_i32(t), dev_i32(l), pol)
            torch.cuda.synchronize()
            assert ctx.device_status() == 0
            ctx.release_groups(groups)
            results.append((t, l, lp.view(np.uint32), pol.cpu().numpy().view(np.uint32)))
    for r in results[1:]:
        for a, b in zip(results[0], r):
            assert np.array_equal(a, b)
    assert np.all(results[0][1] >= 1) and np.all(results[0][1] <= S)
