"""rpo_policy_objective (Eq. 5-7, Eq. 11) on the device against the float64 oracle."""
import numpy as np
import pytest
import torch

import paper_2601_19404_b200 as rpo
import workloads
from oracle import objective as ob
from gpu_util import DEV, make_ctx

pytestmark = pytest.mark.gpu


def _run(ctx, new, old, ref, lens, resp, raw, G, cfg):
    B, S = new.shape
    n_g = B // G
    t = lambda a, dt: None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=dt)).to(DEV)
    R = torch.zeros(B, device=DEV); A = torch.zeros(B, device=DEV); tl = torch.full((B, S), 7.0, device=DEV)
    gobj = torch.zeros(n_g, device=DEV); J = torch.zeros(1, device=DEV)
    ctx.policy_objective(n_g, G, S, t(new, np.float32), t(old, np.float32), t(lens, np.int32), t(raw, np.float32), cfg, R, A, gobj, J,
                         d_logp_ref=t(ref, np.float32), d_resp_lens=t(resp, np.int32), d_token_loss_out=tl)
    torch.cuda.synchronize()
    return R.cpu().numpy(), A.cpu().numpy(), tl.cpu().numpy(), gobj.cpu().numpy(), float(J.item())


@pytest.mark.parametrize("n_groups,G,S", [(1, 1, 1), (3, 4, 7), (16, 8, 128), (5, 64, 300), (32, 6, 33)])
def test_objective_matches_oracle(n_groups, G, S):
    rng = np.random.default_rng(n_groups * 100 + G)
    B = n_groups * G
    lens = rng.integers(0 if B > 1 else 1, S + 1, size=B).astype(np.int32)          # empty suffixes included
    new = (-rng.random((B, S)) * 12).astype(np.float32)
    old = (new + rng.normal(0, 0.3, (B, S))).astype(np.float32)
    ref = (new + rng.normal(0, 0.2, (B, S))).astype(np.float32)
    raw = rng.integers(0, 2, size=B).astype(np.float32)
    resp = (lens + rng.integers(0, 3000, size=B)).astype(np.int32)
    with make_ctx(workloads.SHAPES["tiny"], 1, 1, 32, 4) as ctx:
        for cfg, kw in [(rpo.ObjectiveCfg(0.2, 0.0, 0.01, 0.5, 1.0, True), dict(clip_eps=0.2, beta=0.0)),
                        (rpo.ObjectiveCfg(0.28, 0.04, 0.01, 0.5, 1.0, True), dict(clip_eps=0.28, beta=0.04, logp_ref=ref)),
                        (rpo.ObjectiveCfg(0.2, 0.0, 0.01, 0.5, 1.0, False), dict(clip_eps=0.2, length_shaping=False))]:
            use_ref = ref if cfg.beta != 0 else None
            R, A, tl, gobj, J = _run(ctx, new, old, use_ref, lens, resp, raw, G, cfg)
            o = ob.objective(new.astype(np.float64), old.astype(np.float64), lens, raw, G, alpha=0.01, r_min=0.5, r_max=1.0,
                             resp_lens=resp, **kw)
            assert np.max(np.abs(R - o["rewards"])) < 1e-6
            # the advantage divides by the group's standard deviation: compare where it is not tiny
            assert np.max(np.abs(A - o["advantages"])) < 1e-4 * max(1.0, np.max(np.abs(o["advantages"])))
            assert np.max(np.abs(tl - o["token_loss"])) < 2e-4 * max(1.0, np.max(np.abs(o["token_loss"])))
            assert np.max(np.abs(gobj - o["group_objective"])) < 2e-4
            assert abs(J - o["objective"]) < 2e-4
        # bit-reproducible
        a = _run(ctx, new, old, ref, lens, resp, raw, G, rpo.ObjectiveCfg(0.2, 0.04))
        b = _run(ctx, new, old, ref, lens, resp, raw, G, rpo.ObjectiveCfg(0.2, 0.04))
        assert all(np.array_equal(np.asarray(x).view(np.uint32) if isinstance(x, np.ndarray) else np.float32(x).view(np.uint32),
                                  np.asarray(y).view(np.uint32) if isinstance(y, np.ndarray) else np.float32(y).view(np.uint32))
                   for x, y in zip(a, b))
        if G < 65:
            with pytest.raises(rpo.RpoError):
                z = torch.zeros(130, device=DEV)
                ctx.policy_objective(2, 65, 1, z, z, torch.ones(130, dtype=torch.int32, device=DEV), z, rpo.ObjectiveCfg(), z, z, z, z)
        assert ctx.device_status() == 0


def test_rollout_stage_end_to_end_on_the_tiny_decoder():
    """Algorithm 1's inner loop for two iterations on the tiny fp32 decoder with a synthetic reward."""
    from paper_2601_19404_b200 import experience as ex
    shape = workloads.SHAPES["tiny"]
    rng = np.random.default_rng(5)
    cache = ex.ExperienceCache()
    for q in range(3):
        cache.put(q, rng.integers(0, 1024, 12), rng.integers(0, 1024, 40 + 7 * q))
    G, S = 4, 12
    with make_ctx(shape, 3, G, 120, S, chunk=512) as ctx:
        ctx.init_weights(0, 0.02)
        reward = lambda q, qt, o: float(int(o[-1]) % 2 == 0)                     # stands in for the verifier
        stage = ex.RolloutStage(ctx, cache, G, S, rpo.Sampler(1.0, 0.95, False, -1, 3), reward, L=10, dynamic_factor=0.5, eps=0.5,
                                seed=1, objective_cfg=rpo.ObjectiveCfg(0.2, 0.0, 0.01, 0.5, 1.0, True))
        before = {q: cache.retrieve(q)[1].copy() for q in range(3)}
        for it in range(2):
            res = stage.run([0, 1, 2])
            assert res["tokens"].shape == (3 * G, S) and np.all(res["lens"] == S)
            # first iteration: fixed L = 10; afterwards L = 0.5 * the shortest response of the last group (Eq. 4)
            assert all(0 <= m <= (10 if it == 0 else 0.5 * before[q].size + 1) for q, m in enumerate(res["truncations"]))
            # decode-time and teacher-forced log-probs agree, so every ratio is 1 and the objective is ~0
            assert np.max(np.abs(res["policy_logprobs"] - res["logprobs"])) < 1e-4
            o = ob.objective(res["policy_logprobs"], res["logprobs"], res["lens"], res["raw_rewards"], G, resp_lens=res["resp_lens"])
            assert np.max(np.abs(res["rewards"] - o["rewards"])) < 1e-6 and abs(res["objective"] - o["objective"]) < 1e-4
            for q in range(3):                                                    # the cache now holds one of the new responses
                a = cache.retrieve(q)[1]
                kept = before[q].size - res["truncations"][q]
                assert np.array_equal(a[:kept], before[q][:kept]) and a.size == kept + S
                assert np.array_equal(a[kept:], res["tokens"][q * G + res["chosen"][q]])
                before[q] = a.copy()
        assert ctx.device_status() == 0
