"""Pins of the recurrent-policy oracle (orc_rec_forward_env, orc_rollout_rec).

Referees that are not the oracle's own code: torch.nn.GRUCell / Linear in float64 for the cell, closed forms of saturated
gates, torch.bfloat16 casts for the rounding points of the bf16-operand mode, and a row-by-row re-derivation of the rollout
from the primitive calls across an auto-reset (where the hidden state must restart from zero)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2107_01460_b200 import workloads as wl

REC = ["rec0_tiny_8x8_2p2f_gru64", "rec2_10x10_3p3f_gru64"]


def _split(w, params):
    out, off = {}, 0
    for name, (o, i) in wl.param_shapes(w):
        out[name] = params[off:off + o * i].reshape(o, i); off += o * i
        out["b" + name] = params[off:off + o]; off += o
    assert off == params.size
    return out


def _torch_cell(w, params, obs, h, cast=lambda t: t):
    """The same net written with torch modules' functional forms in float64; `cast` is applied to every operand of a
    product (identity, or a round trip through torch.bfloat16)."""
    F = torch.nn.functional
    p = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in _split(w, params).items()}
    x, h = cast(torch.from_numpy(obs.astype(np.float64))), cast(torch.from_numpy(np.asarray(h, dtype=np.float64)))
    e = cast(F.relu(F.linear(x, cast(p["W1"]), p["bW1"])))
    cell = torch.nn.GRUCell(w["hidden"], w["hidden"]).double()
    with torch.no_grad():
        cell.weight_ih.copy_(cast(p["Wih"])); cell.weight_hh.copy_(cast(p["Whh"]))
        cell.bias_ih.copy_(p["bWih"]); cell.bias_hh.copy_(p["bWhh"])
        h2 = cast(cell(e, h))
        logits = F.linear(h2, cast(p["Wa"]), p["bWa"])
        values = F.linear(h2, cast(p["Wv"]), p["bWv"])[:, 0]
    return logits.numpy(), values.numpy(), h2.numpy()


@pytest.mark.parametrize("name", REC)
def test_cell_against_torch_grucell_in_float64(name):
    w = wl.workload(name)
    cfg = oracle.make_config(w)
    rng = np.random.default_rng(3)
    params = wl.make_params(w, bias_scale=0.3)
    assert params.size == oracle.rec_params_count(cfg)
    N, D, H = w["n_agents"], wl.obs_dim(w), w["hidden"]
    obs = rng.standard_normal((N, D)).astype(np.float32)
    h = rng.standard_normal((N, H)) * 0.7
    lg, v, h2 = oracle.rec_forward_env(cfg, params, obs, h)
    tl, tv, th = _torch_cell(w, params, obs, h)
    assert np.max(np.abs(h2 - th)) < 1e-12 and np.max(np.abs(lg - tl)) < 1e-12 and np.max(np.abs(v - tv)) < 1e-12
    # a transposed weight, a swapped gate block or a missing bias would show: the referee is sensitive to each
    assert np.max(np.abs(th - h)) > 0.05


def test_bf16_operand_mode_rounds_where_torch_bfloat16_casts_do():
    w = wl.workload(REC[0])
    cfg = oracle.make_config(w)
    rng = np.random.default_rng(4)
    params = wl.make_params(w, bias_scale=0.3)
    obs = rng.standard_normal((w["n_agents"], wl.obs_dim(w))).astype(np.float32)
    h = rng.standard_normal((w["n_agents"], w["hidden"])) * 0.7
    cast = lambda t: t.to(torch.float32).to(torch.bfloat16).to(torch.float64)  # noqa: E731
    lg, v, h2 = oracle.rec_forward_env(cfg, params, obs, h, emulate_bf16=True)
    tl, tv, th = _torch_cell(w, params, obs, h, cast)
    assert np.max(np.abs(h2 - th)) < 1e-12 and np.max(np.abs(lg - tl)) < 1e-12 and np.max(np.abs(v - tv)) < 1e-12
    exact = oracle.rec_forward_env(cfg, params, obs, h)[0]
    assert 1e-6 < np.max(np.abs(lg - exact)) < 5e-2


def test_saturated_gates_give_the_closed_forms():
    """Update gate pinned at 1: the state is kept; pinned at 0 with the reset gate at 0: h' = tanh(Win e + bin + 0)."""
    w = wl.workload(REC[0])
    cfg = oracle.make_config(w)
    H, D, N = w["hidden"], wl.obs_dim(w), w["n_agents"]
    rng = np.random.default_rng(5)
    params = wl.make_params(w, bias_scale=0.2)
    P = _split(w, params)  # views into params
    obs = rng.standard_normal((N, D)).astype(np.float32)
    h = rng.standard_normal((N, H)) * 0.5
    P["bWih"][H:2 * H] = 60.0                      # z -> 1
    _, _, h2 = oracle.rec_forward_env(cfg, params, obs, h)
    assert np.max(np.abs(h2 - h)) < 1e-12
    P["bWih"][H:2 * H] = -60.0                     # z -> 0
    P["bWih"][:H] = -60.0                          # r -> 0: the hidden part of the candidate is switched off
    _, _, h2 = oracle.rec_forward_env(cfg, params, obs, h)
    e = np.maximum(obs.astype(np.float64) @ P["W1"].astype(np.float64).T + P["bW1"], 0.0)
    want = np.tanh(e @ P["Wih"][2 * H:].astype(np.float64).T + P["bWih"][2 * H:])
    assert np.max(np.abs(h2 - want)) < 1e-12
    # heads read the NEW state
    lg, v, h2 = oracle.rec_forward_env(cfg, params, obs, h)
    assert np.max(np.abs(lg - (h2 @ P["Wa"].astype(np.float64).T + P["bWa"]))) < 1e-12
    assert np.max(np.abs(v - (h2 @ P["Wv"].astype(np.float64).T + P["bWv"])[:, 0])) < 1e-12


def test_rollout_rows_rederived_from_the_primitives_and_memory_restarts_with_the_episode():
    w = wl.workload(REC[0])
    cfg = oracle.make_config(w)
    params = wl.make_params(w, bias_scale=0.1)
    T, ids = 70, np.array([3, 9], dtype=np.int32)  # longer than the cap of 50: every environment resets inside
    ro, hid = oracle.rollout_rec(cfg, w["seed"], params, T, ids)
    assert ro.dones.sum() >= 2
    N, H = w["n_agents"], w["hidden"]
    for i, e in enumerate(ids):
        s = oracle.env_reset(cfg, w["seed"], int(e), 0)
        h = np.zeros((N, H))
        for t in range(T):
            obs = np.stack([oracle.env_observe(cfg, s, n) for n in range(N)])
            assert np.array_equal(obs, ro.obs[t, i])
            lg, v, h = oracle.rec_forward_env(cfg, params, obs, h)
            assert np.array_equal(lg, ro.logits[t, i]) and np.array_equal(v, ro.values[t, i])
            acts = []
            for n in range(N):
                a, lp, _ = oracle.sample(lg[n], oracle.lib().orc_action_uniform(w["seed"], t, int(e), n))
                acts.append(a)
                assert a == ro.actions[t, i, n] and lp[a] == ro.logp[t, i, n]
            r, d = oracle.env_step(cfg, s, acts)
            assert r == ro.rewards[t, i, 0] and d == ro.dones[t, i]
            if d:
                s = oracle.env_reset(cfg, w["seed"], int(e), s.episode + 1)
                h = np.zeros((N, H))  # the next step must have started from zero memory for the rows above to match
        obs = np.stack([oracle.env_observe(cfg, s, n) for n in range(N)])
        _, v, _ = oracle.rec_forward_env(cfg, params, obs, h)
        assert np.array_equal(v, ro.values[T, i])          # bootstrap on a copy of the state ...
        assert np.array_equal(h, hid[i])                   # ... which is handed back unchanged


def test_replay_equals_free_run_and_two_calls_equal_one():
    w = wl.workload(REC[1])
    cfg = oracle.make_config(w)
    params = wl.make_params(w, bias_scale=0.1)
    ids = np.arange(5, dtype=np.int32)
    whole, hid = oracle.rollout_rec(cfg, w["seed"], params, 40, ids)
    replay, hid2 = oracle.rollout_rec(cfg, w["seed"], params, 40, ids, forced_actions=whole.actions)
    assert np.array_equal(whole.logits, replay.logits) and np.array_equal(hid, hid2)
    a, ha = oracle.rollout_rec(cfg, w["seed"], params, 15, ids)
    b, hb = oracle.rollout_rec(cfg, w["seed"], params, 25, ids, states=a.states, hidden=ha, t_global0=15)
    assert np.array_equal(np.concatenate([a.obs, b.obs]), whole.obs)
    assert np.array_equal(np.concatenate([a.actions, b.actions]), whole.actions)
    assert np.array_equal(np.concatenate([a.values[:15], b.values]), whole.values)
    assert np.array_equal(hb, hid)
    # the memory matters: without it (hidden zeroed between the calls) the second piece differs
    c, _ = oracle.rollout_rec(cfg, w["seed"], params, 25, ids, states=a.states, t_global0=15, forced_actions=b.actions)
    assert not np.array_equal(c.logits, b.logits)
