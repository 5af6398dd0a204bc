"""Group-sharded rollout on the GPU: the gathered batch does not depend on how the groups are
split over ranks (random streams are keyed by the global group id)."""
import numpy as np
import pytest
import torch

import paper_2601_19404_b200 as rpo
from paper_2601_19404_b200 import sharded
import workloads
from gpu_util import DEV, make_ctx, dev_i32

pytestmark = pytest.mark.gpu

TINY = dict(n_layers=2, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688, vocab=1024, rope_base=10000.0,
            rms_eps=1e-6, dtype="fp32")


def test_result_is_independent_of_the_partition():
    G, S = 4, 12
    lens = np.array([40, 17, 64, 33, 25], dtype=np.int32)
    toks, off = workloads.prefix_tokens(lens, TINY["vocab"], seed=4)
    prefixes = [toks[off[g]:off[g + 1]] for g in range(len(lens))]
    smp = rpo.Sampler(1.0, 0.9, False, -1, 7)
    with make_ctx(TINY, len(lens), G, int(lens.max()), S) as ctx:
        ctx.init_weights(seed=0, std=0.02)
        whole = sharded.sharded_rollout(ctx, smp, prefixes, G, S)          # no process group: one rank owns everything
        assert whole["tokens"].shape == (len(lens) * G, S) and np.all(whole["lens"] == S)
        # the same batch as two ranks would compute it, one part after the other on this GPU
        parts = sharded.partition_groups(lens, G, S, 2)
        out = np.zeros_like(whole["tokens"]); lp = np.zeros_like(whole["logprobs"])
        for owned in parts:
            o = np.zeros(len(owned) + 1, dtype=np.int32); o[1:] = np.cumsum(lens[owned])
            t = np.concatenate([prefixes[g] for g in owned]).astype(np.int32)
            groups = ctx.prefill_prefix(dev_i32(t), o, owned.astype(np.int32))
            d_out = torch.zeros((len(owned) * G, S), dtype=torch.int32, device=DEV); d_len = torch.zeros(len(owned) * G, dtype=torch.int32, device=DEV)
            d_lp = torch.zeros((len(owned) * G, S), dtype=torch.float32, device=DEV)
            ctx.decode_suffix(groups, G, S, smp, d_out, d_len, d_lp)
            ctx.release_groups(groups)
            torch.cuda.synchronize()
            for j, g in enumerate(owned):
                out[g * G:(g + 1) * G] = d_out[j * G:(j + 1) * G].cpu().numpy()
                lp[g * G:(g + 1) * G] = d_lp[j * G:(j + 1) * G].cpu().numpy()
        assert np.array_equal(out, whole["tokens"])
        assert np.max(np.abs(lp - whole["logprobs"])) < 1e-5
        assert ctx.device_status() == 0
