"""Pins of the oracle's rollout driver: per-step order, replay, continuation, auto-reset."""
import numpy as np

import oracle
from paper_2107_01460_b200 import workloads as wl


def _setup(idx=0):
    w = wl.workload(idx)
    return w, oracle.make_config(w), wl.make_params(w)


def test_rollout_rows_are_observe_forward_sample_step_in_that_order():
    w, c, params = _setup(0)
    T, env = 60, 3  # longer than the 50-step cap: crosses an auto-reset
    ro = oracle.rollout(c, w["seed"], params, T, [env])
    s = oracle.env_reset(c, w["seed"], env, 0)
    for t in range(T):
        obs = np.stack([oracle.env_observe(c, s, n) for n in range(2)])
        assert np.array_equal(ro.obs[t, 0], obs)
        lg, v = oracle.mlp_forward_env(c, params, obs)
        assert np.array_equal(ro.logits[t, 0], lg) and np.array_equal(ro.values[t, 0], v)
        acts = []
        for n in range(2):
            u = oracle.lib().orc_action_uniform(w["seed"], t, env, n)
            a, lp, m = oracle.sample(lg[n], u)
            acts.append(a)
            assert ro.actions[t, 0, n] == a == ro.own_actions[t, 0, n]
            assert ro.logp[t, 0, n] == lp[a] and ro.margin[t, 0, n] == m
        r, d = oracle.env_step(c, s, acts)
        assert np.all(ro.rewards[t, 0] == r) and ro.dones[t, 0] == d
        if d:
            s = oracle.env_reset(c, w["seed"], env, s.episode + 1)
    obs = np.stack([oracle.env_observe(c, s, n) for n in range(2)])
    assert np.array_equal(ro.values[T, 0], oracle.mlp_forward_env(c, params, obs)[1])
    assert ro.dones.sum() >= 1


def test_replay_of_recorded_actions_reproduces_the_run():
    w, c, params = _setup(0)
    ids = np.arange(6)
    free = oracle.rollout(c, 5, params, 40, ids)
    rep = oracle.rollout(c, 5, params, 40, ids, forced_actions=free.actions)
    env_only = oracle.rollout(c, 5, None, 40, ids, forced_actions=free.actions, compute_mlp=False)
    for a, b in [(free.obs, rep.obs), (free.rewards, rep.rewards), (free.dones, rep.dones),
                 (free.logits, rep.logits), (free.own_actions, rep.own_actions),
                 (free.obs, env_only.obs), (free.rewards, env_only.rewards), (free.dones, env_only.dones)]:
        assert np.array_equal(a, b)


def test_two_calls_continue_like_one():
    w, c, params = _setup(0)
    ids = np.array([1, 9, 4])
    whole = oracle.rollout(c, 2, params, 30, ids)
    first = oracle.rollout(c, 2, params, 18, ids)
    second = oracle.rollout(c, 2, params, 12, ids, states=first.states, t_global0=18)
    assert np.array_equal(whole.actions, np.concatenate([first.actions, second.actions]))
    assert np.array_equal(whole.obs, np.concatenate([first.obs, second.obs]))
    assert np.array_equal(whole.values[18], first.values[18])
    assert np.array_equal(whole.values[30], second.values[12])


def test_envs_are_independent_of_batch_composition():
    w, c, params = _setup(0)
    a = oracle.rollout(c, 0, params, 20, [0, 1, 2, 3])
    b = oracle.rollout(c, 0, params, 20, [3, 1])
    assert np.array_equal(a.obs[:, 3], b.obs[:, 0]) and np.array_equal(a.actions[:, 1], b.actions[:, 1])


def test_centralised_critic_values_are_shared_within_an_env():
    w, c, params = _setup(3)
    ro = oracle.rollout(c, 3, params, 3, [0, 5])
    assert np.all(ro.values == ro.values[:, :, :1])
