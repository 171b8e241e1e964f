"""The host bit selector against what the paper fixes (Section 3.3, Algorithm 2, Section 4.1)."""
import numpy as np
import pytest

from paper_1804_08066_b200.selector import (QNetwork, SarsaBitSelector, WindowQSelector, regression_slope,
                                            reward, smooth_losses)


def test_moving_average_matches_its_closed_form():
    alpha, carry = 0.01, 2.5
    losses = [2.0, 1.5, 1.7, 1.1, 0.9]
    got = smooth_losses(losses, carry, alpha)
    for i in range(5):       # L~_i = (1-a)^i * carry + a * sum_j (1-a)^(i-j) L_j
        want = (1 - alpha) ** (i + 1) * carry + alpha * sum((1 - alpha) ** (i - j) * losses[j] for j in range(i + 1))
        assert got[i] == pytest.approx(want, rel=1e-12)


def test_slope_is_the_least_squares_line_and_reward_has_the_paper_sign():
    v = np.array([3.0, 2.5, 2.7, 2.0, 1.6])
    assert regression_slope(v) == pytest.approx(np.polyfit(np.arange(1, 6), v, 1)[0])
    assert regression_slope(4.0 - 0.25 * np.arange(1, 6)) == pytest.approx(-0.25)
    assert reward(4.0 - 0.25 * np.arange(1, 6), elapsed_ms=50.0, scale=300.0) == pytest.approx(0.25 * 300 / 50)
    assert reward(v, 10.0) > reward(v, 100.0) > 0 > reward(v[::-1], 10.0)


def test_q_network_shape_and_gradient():
    net = QNetwork(5, 10, 7, np.random.default_rng(1))
    assert net.num_parameters() == 5 * 10 + 10 + 10 * 7 + 7 == 137
    x = np.array([0.3, -0.2, 0.5, 0.1, 0.9])
    base = net.q(x)[3]
    eps = 1e-6
    num = np.zeros_like(net.w1)
    for i in range(10):
        for j in range(5):
            net.w1[i, j] += eps
            num[i, j] = (net.q(x)[3] - base) / eps
            net.w1[i, j] -= eps
    before = net.w1.copy()
    net.td_step(x, 3, delta=1.0, lr=1.0)            # w1 += dQ/dw1
    assert np.allclose(net.w1 - before, num, atol=1e-4)
    assert net.q(x)[3] > base                        # moving along the gradient raises Q


def test_widths_change_only_every_period_and_never_decrease():
    sel = SarsaBitSelector(seed=3, epsilon=0.5)
    rng = np.random.default_rng(0)
    bits, prev = [], None
    for m in range(200):
        b = sel.step(m, loss=2.0 * np.exp(-m / 80) + 0.05 * rng.random(), elapsed_ms=30.0)
        assert 2 <= b <= 8
        if prev is not None:
            assert b >= prev
            if m % 5 != 0:
                assert b == prev
        bits.append(b)
        prev = b
    assert bits[0] in (2, 3) and bits[-1] > bits[0]   # exploration raises the width over time
    assert [m for m, _ in sel.history] == list(range(0, 200, 5))


def test_policy_is_epsilon_greedy():
    sel = SarsaBitSelector(seed=5, epsilon=0.1)
    x = np.ones(5)
    keep, more = sel._q_pair(x, 4)
    greedy = 1 if more > keep else 0
    picks = [sel._policy(x, 4) for _ in range(4000)]
    assert abs(np.mean(np.array(picks) != greedy) - 0.1) < 0.02
    assert all(sel._policy(x, 8) == 0 for _ in range(50))      # nothing above the range


def test_sarsa_update_moves_q_towards_the_target():
    sel = SarsaBitSelector(seed=7, epsilon=0.0, lr=0.05)
    for m in range(0, 6):
        sel.step(m, loss=1.0, elapsed_ms=10.0)
    x_prev, n_prev, a_prev = sel.prev
    idx = min(8, n_prev + a_prev) - 2
    q_before = sel.net.q(x_prev)[idx]
    for m in range(6, 11):
        sel.step(m, loss=0.2, elapsed_ms=10.0)       # the loss fell: positive reward
    assert sel.net.q(x_prev)[idx] > q_before


def test_window_selector_stays_in_range_and_learns_from_rewards():
    sel = WindowQSelector(seed=1)
    out = [sel.step(m, loss=1.0 / (1 + m), elapsed_ms=5.0) for m in range(300)]
    assert min(out) >= 1 and max(out) <= 8 and len(set(out)) > 1
    assert np.abs(sel.w).sum() > 0
