"""Pins for the oracle's advantage estimator: none of them restates its backward recursion.

The estimator is defined (Schulman et al., "High-dimensional continuous control using generalized
advantage estimation") as the exponentially weighted sum of temporal-difference residuals,
A_t = sum_l (gamma lambda)^l delta_{t+l}, truncated at episode ends.  The pins evaluate that sum
forwards, or use special cases whose value is a textbook closed form.
"""
import numpy as np
import pytest

from oracle import oracle as O

GAMMA, LAM = 0.99, 0.95          # the paper's baseline hyper-parameters (discount factor, GAE parameter)


def _random_rollout(T, N, seed, p_term=0.05, p_trunc=0.05):
    g = np.random.default_rng(seed)
    reward = g.uniform(0.0, 1.0, (T, N)).astype(np.float32)
    value = g.normal(0.0, 3.0, (T + 1, N)).astype(np.float32)
    flags = ((g.random((T, N)) < p_term).astype(np.uint8) | ((g.random((T, N)) < p_trunc).astype(np.uint8) << 1))
    return reward, value, flags


def _forward_sum(reward, value, flags, gamma, lam, bootstrap):
    """A_t as the forward weighted sum of residuals up to and including the first done step."""
    T, N = reward.shape
    r = reward.astype(np.float64)
    v = value.astype(np.float64)
    adv = np.zeros((T, N))
    for e in range(N):
        for t in range(T):
            w = 1.0
            total = 0.0
            for s in range(t, T):
                term, trunc = flags[s, e] & 1, (flags[s, e] >> 1) & 1
                done = bool(term or trunc)
                rs = r[s, e] + (gamma * v[s, e] if (bootstrap and trunc and not term) else 0.0)
                delta = rs - v[s, e] + (0.0 if done else gamma * v[s + 1, e])
                total += w * delta
                if done:
                    break
                w *= gamma * lam
            adv[t, e] = total
    return adv


@pytest.mark.parametrize("bootstrap", [True, False])
def test_matches_forward_sum_of_residuals(bootstrap):
    reward, value, flags = _random_rollout(32, 40, 1, 0.06, 0.06)
    adv, ret = O.gae(reward, value, flags, GAMMA, LAM, bootstrap)
    ref = _forward_sum(reward, value, flags, GAMMA, LAM, bootstrap)
    np.testing.assert_allclose(adv, ref, atol=1e-10)
    np.testing.assert_allclose(ret, ref + value[:-1].astype(np.float64), atol=1e-10)
    assert (flags == 1).any() and (flags == 2).any()      # both kinds of episode end occur


def test_lambda_one_is_discounted_return_minus_value():
    """lambda = 1, no episode end: A_t = sum_k gamma^k r_{t+k} + gamma^{T-t} V_T - V_t."""
    T, N = 16, 7
    reward, value, _ = _random_rollout(T, N, 2)
    flags = np.zeros((T, N), np.uint8)
    adv, ret = O.gae(reward, value, flags, 0.9, 1.0)
    for t in range(T):
        disc = sum(0.9 ** k * reward[t + k].astype(np.float64) for k in range(T - t))
        disc = disc + 0.9 ** (T - t) * value[T].astype(np.float64)
        np.testing.assert_allclose(ret[t], disc, atol=1e-10)
        np.testing.assert_allclose(adv[t], disc - value[t], atol=1e-10)


def test_lambda_zero_is_the_one_step_residual():
    T, N = 9, 5
    reward, value, _ = _random_rollout(T, N, 3)
    flags = np.zeros((T, N), np.uint8)
    adv, _ = O.gae(reward, value, flags, 0.97, 0.0)
    np.testing.assert_allclose(adv, reward + 0.97 * value[1:].astype(np.float64) - value[:-1], atol=1e-12)


def test_constant_reward_zero_value_is_a_geometric_series():
    T, N = 32, 3
    reward = np.full((T, N), 0.5, np.float32)
    value = np.zeros((T + 1, N), np.float32)
    flags = np.zeros((T, N), np.uint8)
    adv, ret = O.gae(reward, value, flags, GAMMA, LAM)
    x = GAMMA * LAM
    for t in range(T):
        np.testing.assert_allclose(adv[t], 0.5 * (1 - x ** (T - t)) / (1 - x), rtol=1e-12)
    np.testing.assert_allclose(ret, adv)


def test_perfect_value_function_has_zero_advantage():
    """If V satisfies the Bellman equation along the rollout, every residual and so every A_t is 0."""
    T, N = 12, 4
    g = np.random.default_rng(4)
    value = np.zeros((T + 1, N))
    reward = g.uniform(0, 1, (T, N))
    value[T] = g.normal(size=N)
    for t in range(T - 1, -1, -1):
        value[t] = reward[t] + 0.5 * value[t + 1]          # gamma = 1/2: all quantities stay exact-ish
    flags = np.zeros((T, N), np.uint8)
    # fp32 storage of reward/value perturbs the identity by ~1e-7
    adv, _ = O.gae(reward.astype(np.float32), value.astype(np.float32), flags, 0.5, 0.9)
    assert np.abs(adv).max() < 2e-6


def test_episode_end_cuts_the_recursion():
    T, N = 20, 6
    reward, value, _ = _random_rollout(T, N, 5)
    flags = np.zeros((T, N), np.uint8)
    flags[9, :3] = 1                                     # terminated
    flags[9, 3:] = 2                                     # truncated
    a0, _ = O.gae(reward, value, flags, GAMMA, LAM)
    r2, v2 = reward.copy(), value.copy()
    r2[10:] += 5.0                                       # everything after the end of the episode changes
    v2[10:] -= 7.0
    a1, _ = O.gae(r2, v2, flags, GAMMA, LAM)
    np.testing.assert_array_equal(a0[:10], a1[:10])
    assert np.abs(a0[10:] - a1[10:]).min() > 0


def test_terminated_and_truncated_last_step_values():
    """At a terminated step A = r - V; at a truncated one the lost tail is replaced by gamma V."""
    reward = np.array([[0.25, 0.25, 0.25, 0.25]], np.float32)
    value = np.array([[2.0, 2.0, 2.0, 2.0], [9.0, 9.0, 9.0, 9.0]], np.float32)
    flags = np.array([[1, 2, 3, 0]], np.uint8)
    adv, ret = O.gae(reward, value, flags, 0.5, 0.9, bootstrap_truncated=True)
    np.testing.assert_allclose(adv[0], [0.25 - 2.0, 0.25 + 0.5 * 2.0 - 2.0, 0.25 - 2.0, 0.25 + 0.5 * 9.0 - 2.0])
    np.testing.assert_allclose(ret[0], adv[0] + 2.0)
    adv_nb, _ = O.gae(reward, value, flags, 0.5, 0.9, bootstrap_truncated=False)
    np.testing.assert_allclose(adv_nb[0], [0.25 - 2.0, 0.25 - 2.0, 0.25 - 2.0, 0.25 + 0.5 * 9.0 - 2.0])


def test_envs_are_independent_and_layout_is_time_major():
    reward, value, flags = _random_rollout(8, 11, 6)
    adv, ret = O.gae(reward, value, flags, GAMMA, LAM)
    for e in (0, 5, 10):
        a1, r1 = O.gae(reward[:, e:e + 1], value[:, e:e + 1], flags[:, e:e + 1], GAMMA, LAM)
        np.testing.assert_array_equal(a1[:, 0], adv[:, e])
        np.testing.assert_array_equal(r1[:, 0], ret[:, e])
