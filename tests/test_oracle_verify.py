"""Pins for the oracle's draft verification rules."""
import numpy as np

from oracle import cp_head


def test_greedy_acceptance_is_longest_common_prefix():
    d = np.array([[1, 2, 3, 4], [1, 2, 9, 4], [7, 2, 3, 4], [5, 5, 5, 5]])
    b = np.array([[1, 2, 3, 4], [1, 2, 3, 4], [1, 2, 3, 4], [5, 5, 5, 6]])
    assert cp_head.accepted_prefix_greedy(d, b).tolist() == [4, 2, 0, 3]


def test_sampled_acceptance_edge_cases():
    pre = np.log(np.array([[0.5, 0.25, 0.125]]))          # q = 0.5 at every step
    same = np.log(np.full((1, 3), 0.5))
    assert cp_head.accepted_prefix_sampled(pre, same, np.full((1, 3), 0.999)).tolist() == [3]   # p = q: always kept
    low = np.log(np.array([[0.5, 0.1, 0.5]]))              # second token: ratio 0.2
    assert cp_head.accepted_prefix_sampled(pre, low, np.array([[0.9, 0.19, 0.0]])).tolist() == [3]
    assert cp_head.accepted_prefix_sampled(pre, low, np.array([[0.9, 0.21, 0.0]])).tolist() == [1]


def test_first_token_acceptance_rate_is_sum_of_min():
    # draw x ~ q, accept with min(1, p/q): P(accept) = sum_v min(p_v, q_v) (speculative sampling identity)
    rng = np.random.default_rng(0)
    V, draws = 6, 200000
    q = rng.dirichlet(np.ones(V))
    p = rng.dirichlet(np.ones(V))
    x = rng.choice(V, size=draws, p=q)
    acc = cp_head.accepted_prefix_sampled(np.log(q[x])[:, None], np.log(p[x])[:, None], rng.random((draws, 1)))
    assert abs(acc.mean() - np.minimum(p, q).sum()) < 5e-3
