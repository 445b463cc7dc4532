"""Pins of the oracle's MLP (library dense layers as referee), bf16 rounding and the sampler."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2107_01460_b200 import workloads as wl


def _split(w, params):
    out, off = {}, 0
    for name, (o, i) in wl.param_shapes(w):
        out[name] = params[off:off + o * i].reshape(o, i); off += o * i
        out["b_" + name] = params[off:off + o]; off += o
    assert off == params.size
    return out


def _torch_forward(w, params, obs):
    """The same network with torch.nn.functional in float64."""
    F = torch.nn.functional
    p = {k: torch.from_numpy(v.astype(np.float64)) for k, v in _split(w, params).items()}
    x = torch.from_numpy(obs.astype(np.float64))
    h = F.relu(F.linear(F.relu(F.linear(x, p["W1"], p["b_W1"])), p["W2"], p["b_W2"]))
    logits = F.linear(h, p["Wa"], p["b_Wa"])
    if w["net_kind"] == 0:
        values = F.linear(h, p["Wv"], p["b_Wv"])[:, 0]
    else:
        j = x.reshape(1, -1)
        g = F.relu(F.linear(F.relu(F.linear(j, p["C1"], p["b_C1"])), p["C2"], p["b_C2"]))
        values = F.linear(g, p["Cv"], p["b_Cv"])[0].expand(x.shape[0])
    return logits.numpy(), values.numpy()


@pytest.mark.parametrize("idx", range(5))
@pytest.mark.parametrize("bias_scale", [0.0, 0.5])
def test_mlp_matches_torch_float64(idx, bias_scale):
    w = wl.workload(idx)
    c = oracle.make_config(w)
    assert oracle.params_count(c) == wl.params_count(w)
    params = wl.make_params(w, bias_scale=bias_scale)
    s = oracle.env_reset(c, w["seed"], 3, 0)
    obs = np.stack([oracle.env_observe(c, s, n) for n in range(c.n_agents)])
    obs += np.random.default_rng(idx).standard_normal(obs.shape).astype(np.float32) * 0.3  # break sparsity
    lg, v = oracle.mlp_forward_env(c, params, obs)
    lg_t, v_t = _torch_forward(w, params, obs)
    np.testing.assert_allclose(lg, lg_t, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(v, v_t, rtol=1e-12, atol=1e-12)
    if w["net_kind"] == 1:
        assert np.all(v == v[0])


def test_mlp_zero_weights_give_head_biases():
    w = wl.workload(0)
    c = oracle.make_config(w)
    parts = _split(w, np.zeros(wl.params_count(w), dtype=np.float32))
    params = np.zeros(wl.params_count(w), dtype=np.float32)
    # locate the head biases through the shape table
    off = 0
    for name, (o, i) in wl.param_shapes(w):
        off += o * i
        if name == "Wa":
            params[off:off + o] = np.arange(6) * 0.25
        if name == "Wv":
            params[off:off + o] = -1.5
        off += o
    lg, v = oracle.mlp_forward_env(c, params, np.ones((2, 79), dtype=np.float32))
    assert np.array_equal(lg, np.tile(np.arange(6) * 0.25, (2, 1))) and np.all(v == -1.5)
    assert parts["W1"].shape == (64, 79)


def test_mlp_relu_clips_negative_preactivations():
    """Tiny hand network: H=2, one-hot style weights, checks ReLU placement and the [out][in] layout."""
    c = oracle.Config(grid=3, n_agents=1, n_food=1, max_agent_level=1, view_radius=0, episode_cap=5, hidden=2,
                      net_kind=0)
    D = oracle.obs_dim(c)  # 3 + 2 + 1 = 6
    assert D == 6
    W1 = np.zeros((2, D), np.float32); W1[0, 0] = 1.0; W1[1, 1] = -1.0
    W2 = np.array([[1, 0], [2, 1]], np.float32)
    Wa = np.zeros((6, 2), np.float32); Wa[3, 1] = 1.0; Wa[4, 0] = -1.0
    Wv = np.array([[1, 1]], np.float32)
    params = np.concatenate([W1.ravel(), [0.5, 0.25], W2.ravel(), [0, -10], Wa.ravel(), np.zeros(6), Wv.ravel(), [1]]
                            ).astype(np.float32)
    x = np.array([[2, 3, 0, 0, 0, 0]], np.float32)
    # h1 = relu([2+0.5, -3+0.25]) = [2.5, 0]; h2 = relu([2.5, 5-10]) = [2.5, 0]
    lg, v = oracle.mlp_forward_env(c, params, x)
    assert lg[0].tolist() == [0, 0, 0, 0, -2.5, 0] and v[0] == 3.5


def test_bf16_round_matches_torch():
    xs = np.concatenate([np.random.default_rng(0).standard_normal(2000).astype(np.float32) * 10,
                         np.array([0, 1, 1 + 2**-8, 1 + 3 * 2**-8, 0.07, 1e-30, -3.1415927], np.float32)])
    got = np.array([oracle.lib().orc_bf16_round(float(x)) for x in xs], np.float32)
    want = torch.from_numpy(xs).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(got, want)


def test_bf16_emulation_close_to_exact_and_exact_on_bf16_inputs():
    w = wl.workload(1)
    c = oracle.make_config(w)
    params = wl.make_params(w)
    s = oracle.env_reset(c, 1, 0, 0)
    obs = np.stack([oracle.env_observe(c, s, n) for n in range(2)])
    lg, v = oracle.mlp_forward_env(c, params, obs)
    lg_b, v_b = oracle.mlp_forward_env(c, params, obs, emulate_bf16=True)
    assert np.max(np.abs(lg - lg_b)) < 2e-2 and np.max(np.abs(lg - lg_b)) > 0
    assert np.max(np.abs(v - v_b)) < 2e-2


# ---- sampler --------------------------------------------------------------------------------------

def test_equal_logits_give_floor_6u_and_log_sixth():
    for u in [0.0, 0.1, 1 / 6 - 1e-4, 1 / 6 + 1e-4, 0.5, 0.83, 0.9999]:
        a, lp, _ = oracle.sample(np.full(6, 1.7), u)
        assert a == int(math.floor(6 * np.float32(u)))
        np.testing.assert_allclose(lp, -math.log(6), rtol=1e-14)


def test_dominant_logit_wins():
    for k in range(6):
        lg = np.zeros(6); lg[k] = 60.0
        for u in [1e-3, 0.3, 0.99]:
            a, lp, _ = oracle.sample(lg, u)
            assert a == k and abs(lp[k]) < 1e-12


def test_logp_is_log_softmax_and_cdf_boundaries():
    rng = np.random.default_rng(5)
    for _ in range(50):
        lg = rng.standard_normal(6) * 2
        p = torch.softmax(torch.from_numpy(lg), 0).numpy()
        cdf = np.cumsum(p)
        for u in rng.random(20):
            a, lp, m = oracle.sample(lg, float(np.float32(u)))
            uu = float(np.float32(u))
            assert a == int(np.searchsorted(cdf, uu, side="right")) or abs(cdf - uu).min() < 1e-12
            np.testing.assert_allclose(np.exp(lp), p, rtol=1e-12)
            np.testing.assert_allclose(m, np.abs(cdf[:5] - uu).min(), atol=1e-12)
        assert abs(np.exp(lp).sum() - 1) < 1e-12


def test_empirical_frequencies_follow_softmax():
    lg = np.array([0.3, -1.0, 1.2, 0.0, -0.4, 0.8])
    p = np.exp(lg) / np.exp(lg).sum()
    n = 60000
    counts = np.zeros(6)
    for i in range(n):
        u = oracle.lib().orc_action_uniform(99, i, i % 1000, i % 8)
        counts[oracle.sample(lg, u)[0]] += 1
    chi2 = ((counts - n * p) ** 2 / (n * p)).sum()
    assert chi2 < 25.7  # 5 dof, 99.99 % quantile
