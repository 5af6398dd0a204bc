"""Pins of the objective oracle (Eq. 5-7, Eq. 11): closed forms, invariants, brute force."""
import numpy as np
from oracle import objective as ob


def _case(rng, n_groups=3, G=4, S=7):
    B = n_groups * G
    lens = rng.integers(1, S + 1, size=B)
    new = -rng.random((B, S)) * 3; old = new + rng.normal(0, 0.3, (B, S))
    raw = rng.integers(0, 2, size=B).astype(float); raw[0] = 1.0; raw[1] = 0.0
    return new, old, lens, raw


def test_length_aware_reward_closed_forms():
    # a response of exactly the group-mean length keeps half of its reward (sigmoid(0) = 1/2), then the clip
    R = ob.length_aware_rewards([1, 1, 1, 1], [100, 100, 100, 100], 4, alpha=0.01, r_min=0.0, r_max=1.0)
    assert np.allclose(R, 0.5)
    # shorter than average -> larger reward, monotone in the length; bounds are respected
    R = ob.length_aware_rewards([1, 1, 1, 1], [50, 100, 150, 200], 4, alpha=0.01, r_min=0.5, r_max=1.0)
    assert np.all(np.diff(R) <= 0) and R.min() >= 0.5 and R.max() <= 1.0
    unclipped = 1.0 / (1.0 + np.exp(-0.01 * (125.0 - np.array([50, 100, 150, 200]))))
    assert np.allclose(R, np.clip(unclipped, 0.5, 1.0))
    # alpha -> 0 makes every factor 1/2; a zero raw reward stays at the lower bound
    assert np.allclose(ob.length_aware_rewards([1, 1], [10, 500], 2, alpha=0.0, r_min=0.0, r_max=1.0), 0.5)
    assert np.allclose(ob.length_aware_rewards([0, 1], [10, 500], 2, alpha=0.01, r_min=0.5, r_max=1.0)[0], 0.5)


def test_advantages_are_standardised_and_affine_invariant():
    rng = np.random.default_rng(0)
    R = rng.random(12)
    A = ob.group_advantages(R, 4).reshape(3, 4)
    assert np.allclose(A.mean(axis=1), 0) and np.allclose((A ** 2).mean(axis=1), 1)
    assert np.allclose(ob.group_advantages(3.0 * R + 7.0, 4).reshape(3, 4), A)
    assert np.all(ob.group_advantages([0.5, 0.5, 0.5, 0.5], 4) == 0)            # equal rewards: no signal


def test_objective_special_cases():
    rng = np.random.default_rng(1)
    new, old, lens, raw = _case(rng)
    # identical policies: every ratio is 1, token loss = advantage, group objective = mean advantage = 0
    o = ob.objective(new, new, lens, raw, 4, length_shaping=False)
    assert np.allclose(o["group_objective"], 0) and abs(o["objective"]) < 1e-12
    for i in range(len(lens)):
        assert np.allclose(o["token_loss"][i, :lens[i]], o["advantages"][i]) and np.all(o["token_loss"][i, lens[i]:] == 0)
    # a huge clip range removes the clip: l = r A exactly
    o = ob.objective(new, old, lens, raw, 4, clip_eps=1e9, length_shaping=False)
    for i in range(len(lens)):
        assert np.allclose(o["token_loss"][i, :lens[i]], np.exp(new[i, :lens[i]] - old[i, :lens[i]]) * o["advantages"][i])
    # pessimism of the clipped surrogate: never above the unclipped one
    oc = ob.objective(new, old, lens, raw, 4, clip_eps=0.2, length_shaping=False)
    assert np.all(oc["token_loss"] <= o["token_loss"] + 1e-12)
    # positive advantage caps the ratio at 1 + eps, negative advantage floors it at 1 - eps
    one = ob.objective(np.array([[0.0], [0.0]]), np.array([[-1.0], [-1.0]]), [1, 1], [1.0, 0.0], 2, clip_eps=0.2, length_shaping=False)
    assert np.allclose(one["token_loss"][:, 0], [1.2 * 1.0, np.e * -1.0])
    one = ob.objective(np.array([[-1.0], [-1.0]]), np.array([[0.0], [0.0]]), [1, 1], [1.0, 0.0], 2, clip_eps=0.2, length_shaping=False)
    assert np.allclose(one["token_loss"][:, 0], [np.exp(-1.0) * 1.0, 0.8 * -1.0])


def test_kl_term_and_brute_force():
    rng = np.random.default_rng(2)
    new, old, lens, raw = _case(rng, n_groups=2, G=3, S=5)
    ref = new + rng.normal(0, 0.2, new.shape)
    base = ob.objective(new, old, lens, raw, 3, beta=0.0, logp_ref=ref)
    withkl = ob.objective(new, old, lens, raw, 3, beta=0.04, logp_ref=ref)
    assert withkl["objective"] < base["objective"]                               # k3 >= 0, strictly here
    same = ob.objective(new, old, lens, raw, 3, beta=0.04, logp_ref=new)         # KL of a policy with itself
    assert np.allclose(same["token_loss"], base["token_loss"])
    # brute force with python loops
    R = ob.length_aware_rewards(raw, lens, 3, 0.01, 0.5, 1.0)
    total = 0.0
    for g in range(2):
        Rg = R[3 * g:3 * g + 3]; mu = sum(Rg) / 3; sd = (sum((x - mu) ** 2 for x in Rg) / 3) ** 0.5
        acc = 0.0
        for i in range(3):
            b = 3 * g + i; A = (Rg[i] - mu) / sd if sd > 0 else 0.0; s = 0.0
            for j in range(int(lens[b])):
                r = float(np.exp(new[b, j] - old[b, j])); d = ref[b, j] - new[b, j]
                s += min(r * A, min(max(r, 0.8), 1.2) * A) - 0.04 * (float(np.exp(d)) - d - 1.0)
            acc += s / lens[b]
        total += acc / 3
    assert abs(withkl["objective"] - total / 2) < 1e-12
