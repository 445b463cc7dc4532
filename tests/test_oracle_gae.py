"""Pins of the oracle's GAE: the O(T^2) defining sum, closed forms, the effect of a done."""
import numpy as np

import oracle


def _rand(T, E, N, seed, p_done=0.15):
    rng = np.random.default_rng(seed)
    v = rng.standard_normal((T + 1, E, N)).astype(np.float32)
    r = rng.random((T, E, N)).astype(np.float32)
    d = (rng.random((T, E)) < p_done).astype(np.uint8)
    return v, r, d


def test_recurrence_equals_defining_sum():
    for T, E, N in [(1, 2, 2), (7, 3, 2), (16, 4, 3)]:
        for seed in range(3):
            v, r, d = _rand(T, E, N, seed)
            adv, ret = oracle.gae(v, r, d, 0.99, 0.95)
            np.testing.assert_allclose(adv, oracle.gae_bruteforce(v, r, d, 0.99, 0.95), rtol=1e-12, atol=1e-12)
            np.testing.assert_allclose(ret, adv + v[:-1], rtol=0, atol=1e-15)


def test_lambda_zero_is_one_step_td():
    v, r, d = _rand(12, 3, 2, 1)
    adv, _ = oracle.gae(v, r, d, 0.9, 0.0)
    nd = 1.0 - d[:, :, None]
    np.testing.assert_allclose(adv, r.astype(np.float64) + 0.9 * v[1:].astype(np.float64) * nd - v[:-1].astype(np.float64),
                               rtol=1e-13, atol=1e-13)


def test_lambda_one_without_dones_is_discounted_return_minus_value():
    T = 10
    v, r, d = _rand(T, 2, 2, 2, p_done=0.0)
    g = 0.97
    adv, ret = oracle.gae(v, r, d, g, 1.0)
    v = v.astype(np.float64)
    for t in range(T):
        want = sum(g ** l * r[t + l].astype(np.float64) for l in range(T - t)) + g ** (T - t) * v[T] - v[t]
        np.testing.assert_allclose(adv[t], want, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(ret[t], want + v[t], rtol=1e-12, atol=1e-12)


def test_constant_reward_zero_values_geometric_series():
    T, g, lam, rew = 20, 0.99, 0.95, 0.5
    v = np.zeros((T + 1, 1, 1), np.float32)
    r = np.full((T, 1, 1), rew, np.float32)
    d = np.zeros((T, 1), np.uint8)
    adv, _ = oracle.gae(v, r, d, g, lam)
    want = np.array([rew * (1 - (g * lam) ** (T - t)) / (1 - g * lam) for t in range(T)])
    np.testing.assert_allclose(adv[:, 0, 0], want, rtol=1e-12)


def test_done_cuts_bootstrap_and_trace():
    T = 9
    v, r, d = _rand(T, 2, 3, 4, p_done=0.0)
    d[4, 0] = 1
    adv, _ = oracle.gae(v, r, d, 0.99, 0.95)
    v2, r2 = v.copy(), r.copy()
    v2[5:, 0] += 100.0
    r2[5:, 0] -= 7.0
    adv2, _ = oracle.gae(v2, r2, d, 0.99, 0.95)
    assert np.array_equal(adv[:5, 0], adv2[:5, 0])  # nothing after the done leaks back
    np.testing.assert_allclose(adv[4, 0], r[4, 0].astype(np.float64) - v[4, 0], rtol=1e-14)
    assert not np.array_equal(adv[:5, 1], oracle.gae(v2 + 1, r2, d, 0.99, 0.95)[0][:5, 1])


def test_dones_are_shared_by_the_agents_of_an_env():
    v, r, d = _rand(6, 3, 4, 7, p_done=0.4)
    adv, _ = oracle.gae(v, r, d, 0.99, 0.95)
    for n in range(4):
        a1, _ = oracle.gae(v[:, :, n:n + 1], r[:, :, n:n + 1], d, 0.99, 0.95)
        assert np.array_equal(a1[:, :, 0], adv[:, :, n])
