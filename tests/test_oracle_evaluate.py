"""Pins of the oracle's evaluation block: greedy = arg max, episode sums against an independent
recomputation from the rollout's own reward and done arrays, hand-worked episodes."""
import numpy as np

import oracle
from paper_2107_01460_b200 import workloads as wl


def _setup(idx=0):
    w = wl.workload(idx)
    return w, oracle.make_config(w), wl.make_params(w, bias_scale=0.1)


def _episode_sums(rewards, dones):
    """Per environment: count, fp32 sum of returns and sum of lengths of the episodes ending inside
    [0, T), written from the definition (return = sum of the shared step rewards of the episode)."""
    T, n = dones.shape
    cnt = np.zeros(n, np.int32)
    ret = np.zeros(n, np.float32)
    ln = np.zeros(n, np.int32)
    for e in range(n):
        start = 0
        for t in range(T):
            if dones[t, e]:
                g = np.float32(0)
                for k in range(start, t + 1):
                    g = np.float32(g + rewards[k, e, 0])
                ret[e] = np.float32(ret[e] + g)
                ln[e] += t + 1 - start
                cnt[e] += 1
                start = t + 1
    return cnt, ret, ln


def test_greedy_actions_are_the_first_arg_max_of_the_logits():
    w, c, params = _setup(0)
    ev = oracle.evaluate(c, w["seed"], params, 70, np.arange(5))
    assert np.array_equal(ev.actions, np.argmax(ev.logits, axis=-1))
    # a tie goes to the lowest index: all-zero parameters give six equal logits
    ev0 = oracle.evaluate(c, w["seed"], np.zeros_like(params), 10, np.arange(3))
    assert np.all(ev0.actions == 0)


def test_sums_match_a_recomputation_from_the_rollout_under_the_same_actions():
    for idx, T in [(0, 130), (2, 210)]:  # caps 50 and 100: several episodes per environment
        w, c, params = _setup(idx)
        ids = np.array([0, 3, 7, 8])
        ev = oracle.evaluate(c, w["seed"], params, T, ids)
        ro = oracle.rollout(c, w["seed"], None, T, ids, forced_actions=ev.actions, compute_mlp=False, want_obs=False)
        cnt, ret, ln = _episode_sums(ro.rewards, ro.dones)
        assert np.array_equal(ev.ep_count, cnt) and np.array_equal(ev.len_sum, ln)
        assert np.array_equal(ev.ret_sum.view(np.uint32), ret.view(np.uint32))
        assert cnt.min() >= 2
        # the greedy policy's logits are those of the rollout driver on the same states
        full = oracle.rollout(c, w["seed"], params, T, ids, forced_actions=ev.actions, want_obs=False)
        assert np.array_equal(full.logits, ev.logits)
        for a, b in zip(ev.states, ro.states):
            assert bytes(a) == bytes(b)


def test_sampled_evaluation_draws_the_rollouts_actions():
    w, c, params = _setup(0)
    ids = np.arange(4)
    ro = oracle.rollout(c, 9, params, 64, ids, want_obs=False)
    ev = oracle.evaluate(c, 9, params, 64, ids, greedy=False)
    assert np.array_equal(ev.actions, ro.actions)
    cnt, ret, ln = _episode_sums(ro.rewards, ro.dones)
    assert np.array_equal(ev.ep_count, cnt) and np.array_equal(ev.ret_sum, ret) and np.array_equal(ev.len_sum, ln)


def test_hand_worked_episodes():
    """Agents of levels 1 and 2 load the level-3 food of 5 total (reward 3/5), then the level-2 food
    together (2/5): the episode ends at its second step with return 3/5 + 2/5 in binary32; the next
    episode (noops) runs to the cap of 50 with return 0."""
    w, c, params = _setup(0)
    s = oracle.env_reset(c, w["seed"], 0, 0)
    s.agent_r[0], s.agent_c[0], s.agent_level[0] = 3, 2, 1
    s.agent_r[1], s.agent_c[1], s.agent_level[1] = 2, 3, 2
    s.food_r[0], s.food_c[0], s.food_level[0] = 3, 3, 3   # adjacent to both agents
    s.food_r[1], s.food_c[1], s.food_level[1] = 2, 2, 2   # also adjacent to both
    s.total_food_level, s.step, s.episode = 5, 0, 0
    T = 2 + 50 + 5
    forced = np.zeros((T, 1, 2), np.int32)
    forced[0] = 5  # both load: food 0 (3 <= 1+2) and food 1 (2 <= 1+2) are both adjacent to both loaders
    ev = oracle.evaluate(c, w["seed"], params, T, [0], forced_actions=forced, states=[s])
    # both foods go at step 0: reward (3+2)/5 = 1, episode of length 1; then a 50-step episode of noops
    assert ev.ep_count[0] == 2 and ev.len_sum[0] == 1 + 50
    assert ev.ret_sum[0] == np.float32(1.0)
    # one food only: agent 1 alone (level 2) loads; food 1 (level 2) goes, food 0 (level 3) stays
    s2 = oracle.env_reset(c, w["seed"], 0, 0)
    for k in ("agent_r", "agent_c", "agent_level", "food_r", "food_c", "food_level"):
        for i in range(2):
            getattr(s2, k)[i] = getattr(s, k)[i]
    s2.total_food_level, s2.step, s2.episode = 5, 0, 0
    forced2 = np.zeros((52, 1, 2), np.int32)
    forced2[0, 0, 1] = 5
    ev2 = oracle.evaluate(c, w["seed"], params, 52, [0], forced_actions=forced2, states=[s2])
    # the episode runs to its cap (step 50) with return 2/5; the two steps after it belong to an unfinished one
    assert ev2.ep_count[0] == 1 and ev2.len_sum[0] == 50
    assert ev2.ret_sum[0] == np.float32(np.float32(2.0) / np.float32(5.0))


def test_an_unfinished_episode_is_not_counted_and_blocks_continue():
    w, c, params = _setup(0)
    ids = np.arange(3)
    ev = oracle.evaluate(c, w["seed"], params, 20, ids)  # cap 50: nothing can end by the cap in 20 steps
    ro = oracle.rollout(c, w["seed"], None, 20, ids, forced_actions=ev.actions, compute_mlp=False, want_obs=False)
    assert np.array_equal(ev.ep_count, ro.dones.sum(axis=0).astype(np.int32))
    # a second block continues from the first one's states and step counter
    whole = oracle.evaluate(c, w["seed"], params, 90, ids, greedy=False)
    a = oracle.evaluate(c, w["seed"], params, 37, ids, greedy=False)
    b = oracle.evaluate(c, w["seed"], params, 53, ids, greedy=False, states=a.states, t_global0=37)
    assert np.array_equal(whole.actions, np.concatenate([a.actions, b.actions]))
    for x, y in zip(whole.states, b.states):
        assert bytes(x) == bytes(y)
