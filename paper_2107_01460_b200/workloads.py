"""Seeded synthetic workloads: the five rollout configurations and their weights.

This module holds no arithmetic of the method (no environment rule, no network
forward, no sampler, no GAE): only the shape tables and the seeded generator of
the network parameters, so that the CUDA library's tests, the benchmark and the
CPU oracle's tests can all be fed the very same inputs.  It imports numpy only.

The workloads stand in for the level-based foraging tasks the report trains on
(Section 4, "Level-Based Foraging": ``2s-8x8-2p-2f`` and ``15x15-4p-3f``):
same grid sizes, agent and food counts and sight, with a randomly initialised
policy instead of a trained one.
"""
from __future__ import annotations

import numpy as np

N_ACTIONS = 6

# name -> description.  E envs, T steps; precision is the arithmetic the timed
# path uses for that workload ("fp32" SIMT or "bf16" tensor-core operands).
WORKLOADS = {
    "cfg0_tiny_8x8_2p2f_h64": dict(
        grid=8, n_agents=2, n_food=2, max_agent_level=2, view_radius=2, episode_cap=50,
        hidden=64, net_kind=0, n_envs=16, T=32, seed=0, precision="bf16"),
    "cfg1_8x8_2p2f_h128": dict(
        grid=8, n_agents=2, n_food=2, max_agent_level=2, view_radius=2, episode_cap=50,
        hidden=128, net_kind=0, n_envs=1024, T=128, seed=1, precision="bf16"),
    "cfg2_10x10_3p3f_h128": dict(
        grid=10, n_agents=3, n_food=3, max_agent_level=3, view_radius=2, episode_cap=100,
        hidden=128, net_kind=0, n_envs=8192, T=128, seed=2, precision="bf16"),
    "cfg3_15x15_4p5f_mappo_h256": dict(
        grid=15, n_agents=4, n_food=5, max_agent_level=3, view_radius=2, episode_cap=100,
        hidden=256, net_kind=1, n_envs=16384, T=128, seed=3, precision="bf16"),
    "cfg4_20x20_8p8f_h256": dict(
        grid=20, n_agents=8, n_food=8, max_agent_level=3, view_radius=2, episode_cap=100,
        hidden=256, net_kind=0, n_envs=32768, T=64, seed=4, precision="bf16"),
    # Recurrent-policy variants (Section 2: every system has a recurrent version; Section 4: the LBF results are
    # recurrent).  net_kind 2: dense ReLU embedding, one gated recurrent unit of the same width, actor and value heads.
    "rec0_tiny_8x8_2p2f_gru64": dict(
        grid=8, n_agents=2, n_food=2, max_agent_level=2, view_radius=2, episode_cap=50,
        hidden=64, net_kind=2, n_envs=16, T=32, seed=10, precision="bf16"),
    "rec1_8x8_2p2f_gru64": dict(
        grid=8, n_agents=2, n_food=2, max_agent_level=2, view_radius=2, episode_cap=50,
        hidden=64, net_kind=2, n_envs=1024, T=128, seed=11, precision="bf16"),
    "rec2_10x10_3p3f_gru64": dict(
        grid=10, n_agents=3, n_food=3, max_agent_level=3, view_radius=2, episode_cap=100,
        hidden=64, net_kind=2, n_envs=8192, T=128, seed=12, precision="bf16"),
    # Warehouse workloads (Section 4, "Multi-Robot Warehouse"): env_kind 1, or 2 for the variant whose episode ends when
    # two robots get in each other's way; n_food is the number of shelves.  Observations, actions and networks are
    # those of the foraging shapes with the same agent count.
    "wh0_tiny_8x8_2r2s_h64": dict(
        grid=8, n_agents=2, n_food=2, max_agent_level=2, view_radius=2, episode_cap=50, env_kind=1,
        hidden=64, net_kind=0, n_envs=16, T=32, seed=20, precision="bf16"),
    "wh1_10x10_3r3s_h128": dict(
        grid=10, n_agents=3, n_food=3, max_agent_level=3, view_radius=2, episode_cap=100, env_kind=1,
        hidden=128, net_kind=0, n_envs=8192, T=128, seed=21, precision="bf16"),
    "wh2_10x10_3r3s_h128_collisions_end": dict(
        grid=10, n_agents=3, n_food=3, max_agent_level=3, view_radius=2, episode_cap=100, env_kind=2,
        hidden=128, net_kind=0, n_envs=8192, T=128, seed=22, precision="bf16"),
}
WORKLOAD_NAMES = list(WORKLOADS)
GAMMA = 0.99
LAMBDA = 0.95


def workload(name_or_index) -> dict:
    """A copy of one workload description, by name or by index (0..4: the five feed-forward shapes; 5..7: the
    recurrent variants; 8..10: the warehouse workloads)."""
    if isinstance(name_or_index, int):
        name_or_index = WORKLOAD_NAMES[name_or_index]
    w = dict(WORKLOADS[name_or_index])
    w["name"] = name_or_index
    return w


def obs_dim(w: dict) -> int:
    side = 2 * w["view_radius"] + 1
    return 3 * side * side + 2 + w["n_agents"]


def param_shapes(w: dict):
    """(name, (out, in)) of every dense layer, in the order the flat parameter
    array stores them (weight [out][in] then bias [out] for each)."""
    D, H, N = obs_dim(w), w["hidden"], w["n_agents"]
    if w["net_kind"] == 2:  # recurrent: embedding, the cell's input and hidden matrices (gates r, z, n stacked), heads
        return [("W1", (H, D)), ("Wih", (3 * H, H)), ("Whh", (3 * H, H)), ("Wa", (N_ACTIONS, H)), ("Wv", (1, H))]
    layers = [("W1", (H, D)), ("W2", (H, H)), ("Wa", (N_ACTIONS, H))]
    if w["net_kind"] == 0:
        layers += [("Wv", (1, H))]
    else:
        layers += [("C1", (H, N * D)), ("C2", (H, H)), ("Cv", (1, H))]
    return layers


def params_count(w: dict) -> int:
    return sum(o * i + o for _, (o, i) in param_shapes(w))


def make_params(w: dict, seed: int | None = None, bias_scale: float = 0.0) -> np.ndarray:
    """Flat float32 parameters: weights ~ N(0, 1/fan_in); biases 0, or
    N(0, bias_scale^2) for the second test set with non-zero biases."""
    rng = np.random.default_rng(w["seed"] if seed is None else seed)
    parts = []
    for _, (o, i) in param_shapes(w):
        parts.append((rng.standard_normal((o, i)) / np.sqrt(i)).astype(np.float32).ravel())
        b = rng.standard_normal(o) * bias_scale if bias_scale else np.zeros(o)
        parts.append(b.astype(np.float32))
    return np.concatenate(parts)


def sample_env_ids(n_envs: int, head: int, tail: int, rand: int, seed: int = 0) -> np.ndarray:
    """Sorted, distinct environment indices: the first `head`, the last `tail`
    and `rand` seeded-random ones in between (all of them if n_envs is small)."""
    if head + tail + rand >= n_envs:
        return np.arange(n_envs, dtype=np.int32)
    rng = np.random.default_rng(seed)
    mid = rng.choice(np.arange(head, n_envs - tail), size=rand, replace=False)
    ids = np.concatenate([np.arange(head), mid, np.arange(n_envs - tail, n_envs)])
    return np.unique(ids).astype(np.int32)


def shard_first_env(envs_per_rank: int, rank: int) -> int:
    """Global index of a rank's environment 0 when every rank rolls `envs_per_rank` environments
    of one batch of world*envs_per_rank (weak scaling; environments never communicate)."""
    return envs_per_rank * rank
