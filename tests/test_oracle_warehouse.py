"""Pins of the warehouse gridworld of the oracle (orc_wh_reset / orc_wh_observe / orc_wh_step): an independent
restatement of the placement rule, a hand-worked observation, hand-worked transitions for every rule, and invariants over
random-policy runs on every warehouse shape."""
import numpy as np
import pytest

import oracle
from paper_2107_01460_b200 import workloads as wl

WH = ["wh0_tiny_8x8_2r2s_h64", "wh1_10x10_3r3s_h128", "wh2_10x10_3r3s_h128_collisions_end"]


def _cfg(name="wh0_tiny_8x8_2r2s_h64", **over):
    w = wl.workload(name)
    w.update(over)
    return w, oracle.make_config(w)


def _state(cfg, robots, shelves, step=0, episode=0):
    """robots: (r, c, carry) with carry = 0 or 1 + shelf index; shelves: (r, c, status) with 1 idle, 2 requested."""
    s = oracle.EnvState()
    for n, (r, c, k) in enumerate(robots):
        s.agent_r[n], s.agent_c[n], s.agent_level[n] = r, c, k
    for f, (r, c, st) in enumerate(shelves):
        s.food_r[f], s.food_c[f], s.food_level[f] = r, c, st
    s.step, s.episode = step, episode
    return s


def _robots(s, n):
    return [(s.agent_r[i], s.agent_c[i], s.agent_level[i]) for i in range(n)]


def _shelves(s, f):
    return [(s.food_r[i], s.food_c[i], s.food_level[i]) for i in range(f)]


@pytest.mark.parametrize("name", WH)
def test_reset_is_the_stated_placement_rule(name):
    w, cfg = _cfg(name)
    G, N, F = w["grid"], w["n_agents"], w["n_food"]
    L = oracle.lib()

    def draw(env, episode, i):
        key_hi = (w["seed"] >> 32) ^ 0x52534554
        return oracle.philox4x32_10([i // 4, env, episode, 0], [w["seed"] & 0xFFFFFFFF, key_hi])[i % 4]

    for env, episode in [(0, 0), (5, 3), (1234, 1)]:
        s = oracle.wh_reset(cfg, w["seed"], env, episode)
        i = 0
        free_shelf = [c for c in range(G, G * G)]          # rows 1 .. G-1, row-major
        shelves = []
        for k in range(F):
            shelves.append(free_shelf.pop((draw(env, episode, i) * len(free_shelf)) >> 32)); i += 1
        free = [c for c in range(G * G) if c not in shelves]
        robots = []
        for n in range(N):
            robots.append(free.pop((draw(env, episode, i) * len(free)) >> 32)); i += 1
        idle = list(range(F))
        requested = []
        for k in range(max(1, F // 2)):
            requested.append(idle.pop((draw(env, episode, i) * len(idle)) >> 32)); i += 1
        assert [(s.food_r[f] * G + s.food_c[f]) for f in range(F)] == shelves
        assert [(s.agent_r[n] * G + s.agent_c[n]) for n in range(N)] == robots
        assert [f for f in range(F) if s.food_level[f] == 2] == sorted(requested)
        assert all(s.agent_level[n] == 0 for n in range(N)) and s.step == 0 and s.episode == episode
        assert len(set(shelves + robots)) == N + F and min(shelves) >= G


def test_hand_worked_observation():
    w, cfg = _cfg()
    # robot 0 empty-handed at (1,1); robot 1 at (0,2) carrying the requested shelf 1; idle shelf 0 on the ground at (2,1)
    s = _state(cfg, [(1, 1, 0), (0, 2, 2)], [(2, 1, 1), (0, 2, 2)], step=10)
    o = oracle.wh_observe(cfg, s, 0)
    want = np.zeros(79, dtype=np.float32)
    want[12] = 1.0                         # itself, centre of plane 0
    want[1 * 5 + 3] = 2.0                  # robot 1 at dy = -1, dx = +1, carrying
    want[25 + 3 * 5 + 2] = 1.0             # shelf 0 at dy = +1, dx = 0, idle
    want[25 + 1 * 5 + 3] = 2.0             # shelf 1 on robot 1, requested
    for dy in range(-2, 3):
        for dx in range(-2, 3):
            rr, cc, idx = 1 + dy, 1 + dx, 50 + (dy + 2) * 5 + (dx + 2)
            if rr < 0 or cc < 0:
                want[idx] = 1.0            # outside
            elif rr == 0:
                want[idx] = 0.5            # delivery row
    want[75], want[76], want[77] = 1.0, np.float32(10) / np.float32(50), 1.0
    assert np.array_equal(o, want)
    o1 = oracle.wh_observe(cfg, s, 1)
    assert o1[12] == 2.0 and o1[75] == 2.0 and o1[25 + 12] == 2.0 and o1[78] == 1.0


def test_hand_worked_transitions():
    w, cfg = _cfg()
    seed = w["seed"]
    far = (7, 7, 1)

    def step(robots, shelves, acts, kind=1, st=0):
        w2, c2 = _cfg(env_kind=kind)
        s = _state(c2, robots, shelves, step=st)
        r, d = oracle.wh_step(c2, seed, 3, s, acts)
        return _robots(s, 2), _shelves(s, 2), float(r), d

    # an empty-handed robot walks under a shelf on the ground
    rb, sh, r, d = step([(3, 3, 0), (6, 0, 0)], [(3, 4, 1), far], [4, 0])
    assert rb[0] == (3, 4, 0) and sh[0] == (3, 4, 1) and r == 0 and d == 0
    # a carrying robot is stopped by a shelf on the ground (not a robot conflict: the episode goes on even in kind 2)
    rb, sh, r, d = step([(3, 3, 2), (6, 0, 0)], [(3, 4, 1), (3, 3, 2)], [4, 0], kind=2)
    assert rb[0] == (3, 3, 2) and sh[1] == (3, 3, 2) and d == 0
    # pick up: only under a shelf, only empty-handed; the shelf keeps its cell and status
    rb, sh, r, d = step([(3, 4, 0), (6, 0, 0)], [(3, 4, 2), far], [5, 5])
    assert rb[0] == (3, 4, 1) and rb[1] == (6, 0, 0) and sh[0] == (3, 4, 2)
    # a carried shelf moves with its robot
    rb, sh, r, d = step([(3, 4, 1), (6, 0, 0)], [(3, 4, 2), far], [1, 0])
    assert rb[0] == (2, 4, 1) and sh[0] == (2, 4, 2)
    # put down outside the delivery row; refused inside it
    rb, sh, r, d = step([(2, 4, 1), (6, 0, 0)], [(2, 4, 2), far], [5, 0])
    assert rb[0] == (2, 4, 0) and sh[0] == (2, 4, 2)
    rb, sh, r, d = step([(0, 4, 1), (6, 0, 0)], [(0, 4, 1), (7, 7, 2)], [5, 0])
    assert rb[0] == (0, 4, 1) and sh[0] == (0, 4, 1)
    # delivery: a requested shelf carried into row 0 pays 1 to both robots, becomes idle, and the only other idle
    # shelf takes the request (shelf 1 was idle; the delivered one is not eligible)
    rb, sh, r, d = step([(1, 4, 1), (6, 0, 0)], [(1, 4, 2), far], [1, 0])
    assert rb[0] == (0, 4, 1) and sh[0] == (0, 4, 1) and sh[1] == (7, 7, 2) and r == 1.0 and d == 0
    # an idle shelf carried into row 0 pays nothing
    rb, sh, r, d = step([(1, 4, 1), (6, 0, 0)], [(1, 4, 1), (7, 7, 2)], [1, 0])
    assert r == 0.0 and sh[0] == (0, 4, 1) and sh[1] == (7, 7, 2)
    # head-on to the same cell: both stay; it ends the episode only in the variant that says so
    for kind, want_done in ((1, 0), (2, 1)):
        rb, sh, r, d = step([(3, 2, 0), (3, 4, 0)], [far, (6, 6, 2)], [4, 3], kind=kind)
        assert rb == [(3, 2, 0), (3, 4, 0)] and d == want_done
    # following into a cell its occupant is leaving: the follower stays (a conflict), the leader moves
    rb, sh, r, d = step([(3, 2, 0), (3, 3, 0)], [far, (6, 6, 2)], [4, 4], kind=2)
    assert rb == [(3, 2, 0), (3, 4, 0)] and d == 1
    # walls are not conflicts; the cap ends the episode
    rb, sh, r, d = step([(0, 0, 0), (6, 0, 0)], [far, (6, 6, 2)], [1, 0], kind=2)
    assert rb[0] == (0, 0, 0) and d == 0
    rb, sh, r, d = step([(0, 0, 0), (6, 0, 0)], [far, (6, 6, 2)], [0, 0], st=49)
    assert d == 1


def test_two_deliveries_in_one_step_draw_two_replacement_requests_in_robot_order():
    w, cfg = _cfg("wh1_10x10_3r3s_h128", n_food=5)  # five shelves: two requested at all times
    seed = w["seed"]
    s = _state(cfg, [(1, 1, 1), (1, 5, 2), (8, 8, 0)], [(1, 1, 2), (1, 5, 2), (5, 5, 1), (6, 6, 1), (7, 7, 1)], step=4, episode=2)
    r, d = oracle.wh_step(cfg, seed, 9, s, [1, 1, 0])
    assert float(r) == 2.0 and s.total_food_level == 2
    got = [f for f in range(5) if s.food_level[f] == 2]
    idle = [2, 3, 4]
    want = []
    for k in range(2):
        x = oracle.philox4x32_10([k, 9, 2, 4], [seed & 0xFFFFFFFF, (seed >> 32) ^ 0x52455153])[0]
        want.append(idle.pop((x * len(idle)) >> 32))
    assert got == sorted(want) and s.food_level[0] == 1 and s.food_level[1] == 1


@pytest.mark.parametrize("name", WH)
def test_invariants_over_random_policy_runs(name):
    w, cfg = _cfg(name)
    N, F, G = w["n_agents"], w["n_food"], w["grid"]
    rng = np.random.default_rng(1)
    n_req = max(1, F // 2)
    deliveries = conflicts_end = 0
    for env in range(6):
        s = oracle.wh_reset(cfg, w["seed"], env, 0)
        length = 0
        for t in range(400):
            before = _robots(s, N)
            acts = rng.integers(0, 6, N)
            r, d = oracle.wh_step(cfg, w["seed"], env, s, acts)
            length += 1
            rb, sh = _robots(s, N), _shelves(s, F)
            assert len({(a, b) for a, b, _ in rb}) == N                         # robots on distinct cells
            assert len({(a, b) for a, b, _ in sh}) == F                         # at most one shelf per cell
            carried = [k - 1 for _, _, k in rb if k > 0]
            assert len(set(carried)) == len(carried)                            # a shelf rides on one robot at most
            for (a, b, k) in rb:
                assert 0 <= a < G and 0 <= b < G
                if k > 0:
                    assert sh[k - 1][:2] == (a, b)                              # ... and shares its cell
            assert sum(1 for _, _, st in sh if st == 2) == n_req                # the number of requests never changes
            assert all(abs(x[0] - y[0]) + abs(x[1] - y[1]) <= 1 for x, y in zip(before, rb))
            assert float(r) == int(r) and 0 <= r <= min(N, n_req)
            deliveries += int(r)
            for f in range(F):
                if f not in carried:
                    assert sh[f][0] != 0                                        # no shelf is ever left in the delivery row
            if d:
                assert length <= w["episode_cap"]
                conflicts_end += length < w["episode_cap"]
                s = oracle.wh_reset(cfg, w["seed"], env, s.episode + 1)
                length = 0
    assert (conflicts_end > 0) == (w["env_kind"] == 2)
