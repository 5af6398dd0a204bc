"""Host glue of the RPO rollout stage: truncation (Eq. 3-4), prefix construction, epsilon-greedy cache
update (Eq. 10).  No GPU needed."""
import numpy as np
from paper_2601_19404_b200 import experience as ex


def test_truncation_draw_is_uniform_on_0_L_and_clamped():
    rng = np.random.Generator(np.random.PCG64(1))
    draws = np.array([ex.draw_truncation(rng, 7, 1000) for _ in range(16000)])
    assert draws.min() == 0 and draws.max() == 7
    counts = np.bincount(draws, minlength=8)
    assert np.all(np.abs(counts - 2000) < 5 * np.sqrt(2000 * 7 / 8))            # 8 equally likely values
    assert max(ex.draw_truncation(rng, 300, 5) for _ in range(200)) == 5       # never beyond the cached answer
    assert ex.dynamic_L([900, 400, 650], 0.5) == 200                             # L = 0.5 * shortest response


def test_prefix_keeps_everything_for_m_zero_and_drops_the_tail_otherwise():
    q, a = np.array([9, 8], dtype=np.int32), np.arange(10, 20, dtype=np.int32)
    assert ex.build_prefix(q, a, 0).tolist() == [9, 8] + list(range(10, 20))   # NOT the empty python slice a[0:-0]
    assert ex.build_prefix(q, a, 3).tolist() == [9, 8] + list(range(10, 17))
    assert ex.build_prefix(q, a, 10).tolist() == [9, 8] and ex.build_prefix(q, a, 99).tolist() == [9, 8]


def test_epsilon_greedy_selection_frequencies():
    rng = np.random.Generator(np.random.PCG64(2))
    rewards = [0.5, 1.0, 0.7, 1.0]                                               # best = index 1 (first maximum)
    picks = np.array([ex.epsilon_greedy_choice(rng, rewards, 0.25) for _ in range(20000)])
    frac_best = np.mean(picks == 1)
    assert abs(frac_best - 0.25) < 0.015                                         # u <= eps -> the best response
    rest = np.bincount(picks[picks != 1], minlength=4)[[0, 2, 3]]
    assert np.all(np.abs(rest / rest.sum() - 1 / 3) < 0.02)                     # otherwise another one, uniformly
    assert all(ex.epsilon_greedy_choice(rng, rewards, 1.0) == 1 for _ in range(50))
    assert all(ex.epsilon_greedy_choice(rng, rewards, 0.0) != 1 for _ in range(50))
    assert ex.epsilon_greedy_choice(rng, [0.3], 0.0) == 0


def test_cache_put_retrieve_replace():
    c = ex.ExperienceCache()
    c.put("q1", [1, 2], [3, 4, 5]); c.put("q2", [6], [7])
    assert len(c) == 2 and "q1" in c and c.retrieve("q1")[1].tolist() == [3, 4, 5]
    c.put("q1", [1, 2], [9])
    assert len(c) == 2 and c.retrieve("q1")[1].tolist() == [9] and c.retrieve("q1")[0].dtype == np.int32
