"""Pins of the oracle's gridworld: reset, observation, hand-worked transitions, invariants."""
import numpy as np
import pytest

import oracle
from paper_2107_01460_b200 import workloads as wl

NOOP, UP, DOWN, LEFT, RIGHT, LOAD = range(6)


def cfg8(n_agents=2, n_food=2, cap=50):
    return oracle.Config(grid=8, n_agents=n_agents, n_food=n_food, max_agent_level=2, view_radius=2,
                         episode_cap=cap, hidden=64, net_kind=0)


def mk_state(agents, foods, step=0, episode=0, total=None):
    s = oracle.EnvState()
    for i, (r, c, l) in enumerate(agents):
        s.agent_r[i], s.agent_c[i], s.agent_level[i] = r, c, l
    for i, (r, c, l) in enumerate(foods):
        s.food_r[i], s.food_c[i], s.food_level[i] = r, c, l
    s.step, s.episode = step, episode
    s.total_food_level = sum(f[2] for f in foods) if total is None else total
    return s


def agents_of(s, n):
    return [(s.agent_r[i], s.agent_c[i]) for i in range(n)]


FAR_FOODS = [(7, 7, 1), (7, 0, 1)]  # two foods far away from the action


# ---- hand-worked transitions (8x8, two agents) ------------------------------------------------

def test_head_on_same_target_both_stay():
    c = cfg8()
    s = mk_state([(2, 2, 1), (2, 4, 1)], FAR_FOODS)
    r, d = oracle.env_step(c, s, [RIGHT, LEFT])
    assert agents_of(s, 2) == [(2, 2), (2, 4)] and r == 0.0 and d == 0


def test_no_following_into_a_vacated_cell():
    c = cfg8()
    s = mk_state([(2, 2, 1), (2, 3, 1)], FAR_FOODS)
    oracle.env_step(c, s, [RIGHT, RIGHT])
    assert agents_of(s, 2) == [(2, 2), (2, 4)]


def test_no_swap():
    c = cfg8()
    s = mk_state([(2, 2, 1), (2, 3, 1)], FAR_FOODS)
    oracle.env_step(c, s, [RIGHT, LEFT])
    assert agents_of(s, 2) == [(2, 2), (2, 3)]


def test_wall_blocks_on_all_four_sides():
    c = cfg8()
    for pos, a in [((0, 5), UP), ((7, 5), DOWN), ((3, 0), LEFT), ((3, 7), RIGHT)]:
        s = mk_state([(pos[0], pos[1], 1), (5, 5, 1)], [(6, 1, 1), (1, 6, 1)])
        oracle.env_step(c, s, [a, NOOP])
        assert agents_of(s, 2)[0] == pos


def test_free_moves_in_each_direction():
    c = cfg8()
    for a, want in [(UP, (2, 3)), (DOWN, (4, 3)), (LEFT, (3, 2)), (RIGHT, (3, 4)), (NOOP, (3, 3)), (LOAD, (3, 3))]:
        s = mk_state([(3, 3, 1), (6, 6, 1)], FAR_FOODS)
        oracle.env_step(c, s, [a, NOOP])
        assert agents_of(s, 2)[0] == want


def test_food_blocks_a_move():
    c = cfg8()
    s = mk_state([(3, 2, 1), (6, 6, 1)], [(3, 3, 3), (7, 0, 1)])
    oracle.env_step(c, s, [RIGHT, NOOP])
    assert agents_of(s, 2)[0] == (3, 2)


def test_joint_load_collects_and_pays_level_over_total():
    c = cfg8()
    s = mk_state([(3, 2, 1), (2, 3, 2)], [(3, 3, 3), (6, 6, 2)])
    r, d = oracle.env_step(c, s, [LOAD, LOAD])
    assert s.food_level[0] == 0 and s.food_level[1] == 2
    assert r == np.float32(3.0) / np.float32(5.0) and d == 0 and s.step == 1


def test_insufficient_level_collects_nothing():
    c = cfg8()
    s = mk_state([(3, 2, 1), (2, 3, 2)], [(3, 3, 3), (6, 6, 2)])
    r, d = oracle.env_step(c, s, [LOAD, NOOP])
    assert s.food_level[0] == 3 and r == 0.0 and d == 0


def test_diagonal_loader_is_not_adjacent():
    c = cfg8()
    s = mk_state([(3, 2, 1), (2, 2, 2)], [(3, 3, 3), (6, 6, 2)])
    r, _ = oracle.env_step(c, s, [LOAD, LOAD])
    assert s.food_level[0] == 3 and r == 0.0


def test_cell_of_a_food_collected_this_step_is_still_blocked():
    c = cfg8()
    s = mk_state([(3, 2, 1), (2, 3, 1)], [(3, 3, 1), (6, 6, 2)])
    r, _ = oracle.env_step(c, s, [LOAD, DOWN])
    assert s.food_level[0] == 0 and agents_of(s, 2)[1] == (2, 3)
    assert r == np.float32(1.0) / np.float32(3.0)


def test_one_loader_between_two_foods_collects_both():
    c = cfg8()
    s = mk_state([(3, 2, 1), (6, 6, 1)], [(3, 3, 1), (3, 1, 1)])
    r, d = oracle.env_step(c, s, [LOAD, NOOP])
    assert s.food_level[0] == 0 and s.food_level[1] == 0
    assert r == np.float32(2.0) / np.float32(2.0) and d == 1


def test_last_food_ends_the_episode_and_rollout_resets_from_philox():
    c = cfg8()
    seed, env = 11, 5
    s0 = mk_state([(3, 2, 1), (6, 6, 1)], [(3, 3, 1), (0, 0, 0)], step=7, episode=3, total=4)
    forced = np.array([[[LOAD, NOOP]], [[NOOP, NOOP]]], dtype=np.int32)  # T=2, one env
    ro = oracle.rollout(c, seed, None, 2, [env], forced_actions=forced, states=[s0], compute_mlp=False)
    assert ro.dones[:, 0].tolist() == [1, 0]
    assert ro.rewards[0, 0].tolist() == [np.float32(0.25)] * 2
    fresh = oracle.env_reset(c, seed, env, 4)
    fresh_obs = np.stack([oracle.env_observe(c, fresh, n) for n in range(2)])
    assert np.array_equal(ro.obs[1, 0], fresh_obs)  # row after a done shows the new episode
    assert ro.states[0].episode == 4 and ro.states[0].step == 1


def test_cap_truncates():
    c = cfg8(cap=50)
    s = mk_state([(3, 2, 1), (6, 6, 1)], FAR_FOODS, step=48)
    _, d = oracle.env_step(c, s, [NOOP, NOOP])
    assert d == 0 and s.step == 49
    _, d = oracle.env_step(c, s, [NOOP, NOOP])
    assert d == 1 and s.step == 50


def test_three_agents_same_target_all_cancelled_and_independent_mover_goes():
    c = cfg8(n_agents=4)
    s = mk_state([(2, 3, 1), (3, 2, 1), (3, 4, 1), (6, 6, 1)], FAR_FOODS)
    oracle.env_step(c, s, [DOWN, RIGHT, LEFT, UP])
    assert agents_of(s, 4) == [(2, 3), (3, 2), (3, 4), (5, 6)]


# ---- observation -------------------------------------------------------------------------------

def test_observation_hand_worked_corner():
    c = cfg8()
    s = mk_state([(0, 0, 1), (1, 2, 2)], [(2, 0, 3), (7, 7, 1)], step=0)
    o = oracle.env_observe(c, s, 0)
    want = np.zeros(79, dtype=np.float32)
    want[12] = 1  # own level in the centre of the agent plane
    want[19] = 2  # agent 1 at (dy,dx)=(+1,+2)
    want[25 + 22] = 3  # food at (dy,dx)=(+2,0)
    for i in [0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 15, 16, 20, 21]:
        want[50 + i] = 1  # two rows above and two columns left are outside
    want[75], want[76], want[77], want[78] = 1, 0, 1, 0
    assert np.array_equal(o, want)
    o1 = oracle.env_observe(c, s, 1)
    assert o1[12] == 2 and o1[12 - 5 - 2] == 1  # agent 0 seen at (dy,dx)=(-1,-2)
    assert o1[25 + (1 + 2) * 5 + (-2 + 2)] == 3  # food at (dy,dx)=(+1,-2)
    assert o1[75] == 2 and o1[77] == 0 and o1[78] == 1
    assert o1[50:75].sum() == 5  # one row above the grid


def test_observation_step_fraction_and_gone_food():
    c = cfg8()
    s = mk_state([(4, 4, 1), (4, 5, 2)], [(3, 4, 0), (5, 4, 2)], step=7, total=4)
    o = oracle.env_observe(c, s, 0)
    assert o[76] == np.float32(7) / np.float32(50)
    assert o[25 + 1 * 5 + 2] == 0  # collected food is invisible
    assert o[25 + 3 * 5 + 2] == 2
    assert o[50:75].sum() == 0


@pytest.mark.parametrize("idx", range(5))
def test_observation_invariants_on_resets(idx):
    w = wl.workload(idx)
    c = oracle.make_config(w)
    D, G, N = oracle.obs_dim(c), c.grid, c.n_agents
    assert D == wl.obs_dim(w)
    for env in range(40):
        s = oracle.env_reset(c, w["seed"], env, 0)
        for n in range(N):
            o = oracle.env_observe(c, s, n)
            r, cc = s.agent_r[n], s.agent_c[n]
            rows_in = sum(0 <= r + d < G for d in range(-2, 3))
            cols_in = sum(0 <= cc + d < G for d in range(-2, 3))
            assert o[50:75].sum() == 25 - rows_in * cols_in
            assert o[12] == s.agent_level[n] == o[75]
            assert o[77:77 + N].sum() == 1 and o[77 + n] == 1


# ---- reset --------------------------------------------------------------------------------------

def _reset_draws(seed, env, episode, count):
    key = [seed & 0xFFFFFFFF, ((seed >> 32) ^ 0x52534554) & 0xFFFFFFFF]
    out = []
    for i in range(count):
        out.append(oracle.philox4x32_10([i // 4, env, episode, 0], key)[i % 4])
    return out


@pytest.mark.parametrize("grid,n_agents,n_food,lmax", [(3, 2, 2, 2), (3, 4, 5, 3), (8, 2, 2, 2), (20, 8, 8, 3)])
def test_reset_equals_pop_from_free_list(grid, n_agents, n_food, lmax):
    """Independent restatement: keep the free cells in a sorted list and pop index r."""
    c = oracle.Config(grid=grid, n_agents=n_agents, n_food=n_food, max_agent_level=lmax, view_radius=2,
                      episode_cap=50, hidden=8, net_kind=0)
    for seed, env, ep in [(0, 0, 0), (7, 3, 1), (2**40 + 5, 1000, 17)]:
        d = _reset_draws(seed, env, ep, 2 * (n_agents + n_food))
        al = [1 + (d[i] * lmax >> 32) for i in range(n_agents)]
        S = sum(al)
        fl = [1 + (d[n_agents + i] * S >> 32) for i in range(n_food)]
        free = list(range(grid * grid))
        cells = []
        for k in range(n_agents + n_food):
            r = d[n_agents + n_food + k] * (grid * grid - k) >> 32
            cells.append(free.pop(r))
        s = oracle.env_reset(c, seed, env, ep)
        assert [s.agent_level[i] for i in range(n_agents)] == al
        assert [s.food_level[i] for i in range(n_food)] == fl
        got = [s.agent_r[i] * grid + s.agent_c[i] for i in range(n_agents)]
        got += [s.food_r[i] * grid + s.food_c[i] for i in range(n_food)]
        assert got == cells
        assert s.total_food_level == sum(fl) and s.step == 0 and s.episode == ep


def test_reset_invariants_and_uniformity():
    c = cfg8()
    G, n = 8, 20000
    cell_counts = np.zeros((4, G * G))
    lvl_counts = np.zeros(3)
    for env in range(n):
        s = oracle.env_reset(c, 123, env, env % 7)
        cells = [s.agent_r[i] * G + s.agent_c[i] for i in range(2)] + [s.food_r[i] * G + s.food_c[i] for i in range(2)]
        assert len(set(cells)) == 4 and all(0 <= x < G * G for x in cells)
        S = s.agent_level[0] + s.agent_level[1]
        assert all(1 <= s.agent_level[i] <= 2 for i in range(2))
        assert all(1 <= s.food_level[i] <= S for i in range(2))
        for k, x in enumerate(cells):
            cell_counts[k, x] += 1
        lvl_counts[s.agent_level[0]] += 1
    # chi-square against the uniform law; 63 dof, 99.99% quantile is ~114
    for k in range(4):
        chi2 = ((cell_counts[k] - n / 64) ** 2 / (n / 64)).sum()
        assert chi2 < 130, (k, chi2)
    assert abs(lvl_counts[1] / n - 0.5) < 0.02


# ---- invariants over random-policy runs -------------------------------------------------------

@pytest.mark.parametrize("idx", range(5))
def test_step_invariants_under_random_actions(idx):
    w = wl.workload(idx)
    c = oracle.make_config(w)
    N, F, G, cap = c.n_agents, c.n_food, c.grid, c.episode_cap
    rng = np.random.default_rng(idx)
    collected_episodes = 0
    for env in range(12):
        s = oracle.env_reset(c, w["seed"], env, 0)
        ep_reward = np.float64(0)
        for _ in range(3 * cap):
            before = oracle.EnvState.from_buffer_copy(s)
            acts = rng.integers(0, 6, N)
            # bias towards loading next to food so that collections do happen
            for n in range(N):
                for f in range(F):
                    if s.food_level[f] > 0 and abs(s.agent_r[n] - s.food_r[f]) + abs(s.agent_c[n] - s.food_c[f]) == 1:
                        if rng.random() < 0.7:
                            acts[n] = LOAD
            r, d = oracle.env_step(c, s, acts)
            pos = agents_of(s, N)
            assert len(set(pos)) == N and all(0 <= a < G and 0 <= b < G for a, b in pos)
            for n in range(N):
                assert abs(pos[n][0] - before.agent_r[n]) + abs(pos[n][1] - before.agent_c[n]) <= 1
            gone = 0
            for f in range(F):
                if s.food_level[f] > 0:
                    assert (s.food_r[f], s.food_c[f]) not in pos
                    assert s.food_level[f] == before.food_level[f]
                elif before.food_level[f] > 0:
                    load = sum(before.agent_level[n] for n in range(N) if acts[n] == LOAD and
                               abs(before.agent_r[n] - s.food_r[f]) + abs(before.agent_c[n] - s.food_c[f]) == 1)
                    assert load >= before.food_level[f]
                    gone += before.food_level[f]
            assert r == (np.float32(gone) / np.float32(s.total_food_level) if gone else 0.0)
            assert 0.0 <= r <= 1.0
            ep_reward += r
            assert s.step == before.step + 1 <= cap
            left = sum(s.food_level[f] > 0 for f in range(F))
            assert d == int(left == 0 or s.step >= cap)
            if d:
                if left == 0:
                    assert abs(ep_reward - 1.0) < 1e-5
                    collected_episodes += 1
                else:
                    assert s.step == cap and ep_reward < 1.0 + 1e-5
                s = oracle.env_reset(c, w["seed"], env, s.episode + 1)
                ep_reward = np.float64(0)
    if idx < 2:
        assert collected_episodes > 0
