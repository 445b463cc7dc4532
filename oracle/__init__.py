"""ctypes front end of the CPU oracle (``mava_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg; the CUDA library and its Python binding never
import this package, and this package never imports them.

All arithmetic of the rollout, the evaluation block and GAE lives in the C file; this
module only builds the shared object (``gcc``) and marshals numpy arrays.  The update
block (multi-agent PPO loss, its gradient, Adam) is ``oracle/ppo.py``, plain numpy in float64.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mava_oracle.c")
_LIB = os.path.join(_HERE, "libmava_oracle.so")

MAX_AGENTS = 8
MAX_FOOD = 8
N_ACTIONS = 6


def build(force: bool = False) -> str:
    """Compile the oracle with gcc when the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-std=c11", "-O2", "-Wall", "-Wextra", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


class Config(C.Structure):
    _fields_ = [
        ("grid", C.c_int32),
        ("n_agents", C.c_int32),
        ("n_food", C.c_int32),
        ("max_agent_level", C.c_int32),
        ("view_radius", C.c_int32),
        ("episode_cap", C.c_int32),
        ("hidden", C.c_int32),
        ("net_kind", C.c_int32),
        ("env_kind", C.c_int32),
    ]


class EnvState(C.Structure):
    _fields_ = [
        ("agent_r", C.c_int32 * MAX_AGENTS),
        ("agent_c", C.c_int32 * MAX_AGENTS),
        ("agent_level", C.c_int32 * MAX_AGENTS),
        ("food_r", C.c_int32 * MAX_FOOD),
        ("food_c", C.c_int32 * MAX_FOOD),
        ("food_level", C.c_int32 * MAX_FOOD),
        ("step", C.c_int32),
        ("episode", C.c_int32),
        ("total_food_level", C.c_int32),
    ]


def make_config(workload: dict) -> Config:
    """Config from a workload description (keys named like the struct fields)."""
    return Config(**{name: int(workload.get(name, 0)) for name, _ in Config._fields_})


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u32p = C.POINTER(C.c_uint32)
        L.orc_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.orc_philox4x32_10.restype = None
        L.orc_bounded.argtypes = [C.c_uint32, C.c_uint32]
        L.orc_bounded.restype = C.c_uint32
        L.orc_uniform24.argtypes = [C.c_uint32]
        L.orc_uniform24.restype = C.c_float
        L.orc_action_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32]
        L.orc_action_uniform.restype = C.c_float
        L.orc_obs_dim.argtypes = [C.POINTER(Config)]
        L.orc_obs_dim.restype = C.c_int32
        L.orc_params_count.argtypes = [C.POINTER(Config)]
        L.orc_params_count.restype = C.c_int64
        L.orc_bf16_round.argtypes = [C.c_float]
        L.orc_bf16_round.restype = C.c_float
        L.orc_env_reset.argtypes = [C.POINTER(Config), C.c_uint64, C.c_int32, C.c_int32, C.POINTER(EnvState)]
        L.orc_env_reset.restype = None
        L.orc_env_observe.argtypes = [C.POINTER(Config), C.POINTER(EnvState), C.c_int32, C.c_void_p]
        L.orc_env_observe.restype = None
        L.orc_env_step.argtypes = [C.POINTER(Config), C.POINTER(EnvState), C.c_void_p, C.POINTER(C.c_float),
                                   C.POINTER(C.c_uint8)]
        L.orc_env_step.restype = None
        L.orc_wh_reset.argtypes = [C.POINTER(Config), C.c_uint64, C.c_int32, C.c_int32, C.POINTER(EnvState)]
        L.orc_wh_reset.restype = None
        L.orc_wh_observe.argtypes = [C.POINTER(Config), C.POINTER(EnvState), C.c_int32, C.c_void_p]
        L.orc_wh_observe.restype = None
        L.orc_wh_step.argtypes = [C.POINTER(Config), C.c_uint64, C.c_int32, C.POINTER(EnvState), C.c_void_p,
                                  C.POINTER(C.c_float), C.POINTER(C.c_uint8)]
        L.orc_wh_step.restype = None
        L.orc_mlp_forward_env.argtypes = [C.POINTER(Config), C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_mlp_forward_env.restype = None
        L.orc_sample.argtypes = [C.c_void_p, C.c_float, C.POINTER(C.c_int32), C.c_void_p, C.POINTER(C.c_double)]
        L.orc_sample.restype = None
        L.orc_rollout.argtypes = [
            C.POINTER(Config), C.c_uint64, C.c_void_p, C.c_int, C.c_int, C.c_int32, C.c_void_p, C.c_int32,
            C.c_int32, C.c_int32, C.c_uint32, C.POINTER(EnvState), C.c_void_p,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p,
        ]
        L.orc_rollout.restype = C.c_int
        L.orc_evaluate.argtypes = [
            C.POINTER(Config), C.c_uint64, C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_int32, C.c_uint32,
            C.POINTER(EnvState), C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
        ]
        L.orc_evaluate.restype = C.c_int
        L.orc_rec_params_count.argtypes = [C.POINTER(Config)]
        L.orc_rec_params_count.restype = C.c_int64
        L.orc_rec_forward_env.argtypes = [C.POINTER(Config), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_rec_forward_env.restype = None
        L.orc_rollout_rec.argtypes = [
            C.POINTER(Config), C.c_uint64, C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_int32, C.c_uint32,
            C.POINTER(EnvState), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
        ]
        L.orc_rollout_rec.restype = C.c_int
        L.orc_gae.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_double,
                              C.c_double, C.c_void_p, C.c_void_p]
        L.orc_gae.restype = None
        L.orc_gae_bruteforce.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_double, C.c_double, C.c_void_p]
        L.orc_gae_bruteforce.restype = None
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def philox4x32_10(ctr, key):
    c = (C.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (C.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    out = (C.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, out)
    return [int(x) for x in out]


def obs_dim(cfg: Config) -> int:
    return int(lib().orc_obs_dim(C.byref(cfg)))


def params_count(cfg: Config) -> int:
    return int(lib().orc_params_count(C.byref(cfg)))


def env_reset(cfg: Config, seed: int, env: int, episode: int) -> EnvState:
    s = EnvState()
    lib().orc_env_reset(C.byref(cfg), C.c_uint64(seed), env, episode, C.byref(s))
    return s


def wh_reset(cfg: Config, seed: int, env: int, episode: int) -> EnvState:
    """Start of a warehouse episode (see orc_wh_reset for how the state's fields are used)."""
    s = EnvState()
    lib().orc_wh_reset(C.byref(cfg), C.c_uint64(seed), env, episode, C.byref(s))
    return s


def wh_observe(cfg: Config, state: EnvState, agent: int) -> np.ndarray:
    out = np.empty(obs_dim(cfg), dtype=np.float32)
    lib().orc_wh_observe(C.byref(cfg), C.byref(state), agent, _ptr(out))
    return out


def wh_step(cfg: Config, seed: int, env: int, state: EnvState, actions):
    """Advance a warehouse `state` in place; returns (reward, done)."""
    a = np.ascontiguousarray(actions, dtype=np.int32)
    assert a.size == cfg.n_agents
    r = C.c_float()
    d = C.c_uint8()
    lib().orc_wh_step(C.byref(cfg), C.c_uint64(seed), env, C.byref(state), _ptr(a), C.byref(r), C.byref(d))
    return np.float32(r.value), int(d.value)


def initial_state(cfg: Config, seed: int, env: int, episode: int = 0) -> EnvState:
    """Start-of-episode state of the workload family the config names."""
    return env_reset(cfg, seed, env, episode) if cfg.env_kind == 0 else wh_reset(cfg, seed, env, episode)


def env_observe(cfg: Config, state: EnvState, agent: int) -> np.ndarray:
    out = np.empty(obs_dim(cfg), dtype=np.float32)
    lib().orc_env_observe(C.byref(cfg), C.byref(state), agent, _ptr(out))
    return out


def env_step(cfg: Config, state: EnvState, actions):
    """Advance ``state`` in place; returns (reward, done)."""
    a = np.ascontiguousarray(actions, dtype=np.int32)
    assert a.size == cfg.n_agents
    r = C.c_float()
    d = C.c_uint8()
    lib().orc_env_step(C.byref(cfg), C.byref(state), _ptr(a), C.byref(r), C.byref(d))
    return np.float32(r.value), int(d.value)


def mlp_forward_env(cfg: Config, params: np.ndarray, obs: np.ndarray, emulate_bf16: bool = False):
    """obs [N][D] float32 -> (logits [N][6] float64, values [N] float64)."""
    p = np.ascontiguousarray(params, dtype=np.float32)
    o = np.ascontiguousarray(obs, dtype=np.float32)
    assert p.size == params_count(cfg) and o.size == cfg.n_agents * obs_dim(cfg)
    logits = np.empty((cfg.n_agents, N_ACTIONS), dtype=np.float64)
    values = np.empty(cfg.n_agents, dtype=np.float64)
    lib().orc_mlp_forward_env(C.byref(cfg), _ptr(p), _ptr(o), int(emulate_bf16), _ptr(logits), _ptr(values))
    return logits, values


def sample(logits, u: float):
    """(action, logp[6], margin) for six logits and a uniform u in [0,1)."""
    lg = np.ascontiguousarray(logits, dtype=np.float64)
    assert lg.size == N_ACTIONS
    a = C.c_int32()
    m = C.c_double()
    lp = np.empty(N_ACTIONS, dtype=np.float64)
    lib().orc_sample(_ptr(lg), C.c_float(u), C.byref(a), _ptr(lp), C.byref(m))
    return int(a.value), lp, float(m.value)


@dataclass
class Rollout:
    obs: np.ndarray | None
    actions: np.ndarray
    own_actions: np.ndarray | None
    logp: np.ndarray | None
    values: np.ndarray | None
    rewards: np.ndarray
    dones: np.ndarray
    logits: np.ndarray | None
    margin: np.ndarray | None
    states: list


def rollout(cfg: Config, seed: int, params, T: int, env_ids, *, forced_actions=None, states=None,
            t_global0: int = 0, emulate_bf16: bool = False, compute_mlp: bool = True,
            want_obs: bool = True) -> Rollout:
    """Roll the listed environments for T steps (arrays are [T][len(env_ids)][N]...).

    ``states`` defaults to the episode-0 reset of every listed environment.
    """
    env_ids = np.ascontiguousarray(env_ids, dtype=np.int32)
    n = int(env_ids.size)
    N, D = cfg.n_agents, obs_dim(cfg)
    if states is None:
        states = [initial_state(cfg, seed, int(e), 0) for e in env_ids]
    st = (EnvState * n)(*states)
    fa = None
    if forced_actions is not None:
        fa = np.ascontiguousarray(forced_actions, dtype=np.int32)
        assert fa.shape == (T, n, N)
    p = None
    if compute_mlp:
        p = np.ascontiguousarray(params, dtype=np.float32)
        assert p.size == params_count(cfg)
    obs = np.empty((T, n, N, D), dtype=np.float32) if want_obs else None
    actions = np.empty((T, n, N), dtype=np.int32)
    rewards = np.empty((T, n, N), dtype=np.float32)
    dones = np.empty((T, n), dtype=np.uint8)
    own = logp = values = logits = margin = None
    if compute_mlp:
        own = np.empty((T, n, N), dtype=np.int32)
        logp = np.empty((T, n, N), dtype=np.float64)
        values = np.empty((T + 1, n, N), dtype=np.float64)
        logits = np.empty((T, n, N, N_ACTIONS), dtype=np.float64)
        margin = np.empty((T, n, N), dtype=np.float64)
    rc = lib().orc_rollout(C.byref(cfg), C.c_uint64(seed), _ptr(p), int(emulate_bf16), int(compute_mlp), n,
                           _ptr(env_ids), n, 0, T, t_global0, st, _ptr(fa), _ptr(obs), _ptr(actions), _ptr(own),
                           _ptr(logp), _ptr(values), _ptr(rewards), _ptr(dones), _ptr(logits), _ptr(margin))
    if rc != 0:
        raise ValueError("orc_rollout rejected its arguments")
    return Rollout(obs, actions, own, logp, values, rewards, dones, logits, margin, list(st))


def rec_params_count(cfg: Config) -> int:
    return int(lib().orc_rec_params_count(C.byref(cfg)))


def rec_forward_env(cfg: Config, params: np.ndarray, obs: np.ndarray, hidden: np.ndarray, emulate_bf16: bool = False):
    """Recurrent policy, one environment, one step: obs [N][D] float32, hidden [N][H] float64 ->
    (logits [N][6], values [N], new hidden [N][H]), all float64."""
    p = np.ascontiguousarray(params, dtype=np.float32)
    o = np.ascontiguousarray(obs, dtype=np.float32)
    h = np.array(hidden, dtype=np.float64, order="C", copy=True)
    assert p.size == rec_params_count(cfg) and o.size == cfg.n_agents * obs_dim(cfg) and h.shape == (cfg.n_agents, cfg.hidden)
    logits = np.empty((cfg.n_agents, N_ACTIONS), dtype=np.float64)
    values = np.empty(cfg.n_agents, dtype=np.float64)
    lib().orc_rec_forward_env(C.byref(cfg), _ptr(p), _ptr(o), _ptr(h), int(emulate_bf16), _ptr(logits), _ptr(values))
    return logits, values, h


def rollout_rec(cfg: Config, seed: int, params, T: int, env_ids, *, forced_actions=None, states=None, hidden=None,
                t_global0: int = 0, emulate_bf16: bool = False, want_obs: bool = True):
    """The rollout with the recurrent policy; returns (Rollout, hidden [n][N][H] float64 after the run).  `hidden`
    defaults to zeros (every environment at the start of an episode)."""
    env_ids = np.ascontiguousarray(env_ids, dtype=np.int32)
    n = int(env_ids.size)
    N, D, H = cfg.n_agents, obs_dim(cfg), cfg.hidden
    if states is None:
        states = [initial_state(cfg, seed, int(e), 0) for e in env_ids]
    st = (EnvState * n)(*states)
    hid = np.zeros((n, N, H), dtype=np.float64) if hidden is None else np.array(hidden, dtype=np.float64, order="C", copy=True)
    assert hid.shape == (n, N, H)
    fa = None
    if forced_actions is not None:
        fa = np.ascontiguousarray(forced_actions, dtype=np.int32)
        assert fa.shape == (T, n, N)
    p = np.ascontiguousarray(params, dtype=np.float32)
    assert p.size == rec_params_count(cfg)
    obs = np.empty((T, n, N, D), dtype=np.float32) if want_obs else None
    actions = np.empty((T, n, N), dtype=np.int32)
    own = np.empty((T, n, N), dtype=np.int32)
    logp = np.empty((T, n, N), dtype=np.float64)
    values = np.empty((T + 1, n, N), dtype=np.float64)
    rewards = np.empty((T, n, N), dtype=np.float32)
    dones = np.empty((T, n), dtype=np.uint8)
    logits = np.empty((T, n, N, N_ACTIONS), dtype=np.float64)
    margin = np.empty((T, n, N), dtype=np.float64)
    rc = lib().orc_rollout_rec(C.byref(cfg), C.c_uint64(seed), _ptr(p), int(emulate_bf16), n, _ptr(env_ids), T, t_global0,
                               st, _ptr(hid), _ptr(fa), _ptr(obs), _ptr(actions), _ptr(own), _ptr(logp), _ptr(values),
                               _ptr(rewards), _ptr(dones), _ptr(logits), _ptr(margin))
    if rc != 0:
        raise ValueError("orc_rollout_rec rejected its arguments")
    return Rollout(obs, actions, own, logp, values, rewards, dones, logits, margin, list(st)), hid


@dataclass
class Evaluation:
    ep_count: np.ndarray   # [n] int32
    ret_sum: np.ndarray    # [n] float32
    len_sum: np.ndarray    # [n] int32
    actions: np.ndarray    # [T][n][N] int32
    logits: np.ndarray     # [T][n][N][6] float64
    states: list


def evaluate(cfg: Config, seed: int, params, T: int, env_ids, *, greedy: bool = True, forced_actions=None,
             states=None, t_global0: int = 0, emulate_bf16: bool = False) -> Evaluation:
    """An evaluation block of T steps over the listed environments (see orc_evaluate)."""
    env_ids = np.ascontiguousarray(env_ids, dtype=np.int32)
    n = int(env_ids.size)
    N = cfg.n_agents
    if states is None:
        states = [initial_state(cfg, seed, int(e), 0) for e in env_ids]
    st = (EnvState * n)(*states)
    fa = None
    if forced_actions is not None:
        fa = np.ascontiguousarray(forced_actions, dtype=np.int32)
        assert fa.shape == (T, n, N)
    p = np.ascontiguousarray(params, dtype=np.float32)
    assert p.size == params_count(cfg)
    ep = np.empty(n, dtype=np.int32)
    rs = np.empty(n, dtype=np.float32)
    ls = np.empty(n, dtype=np.int32)
    actions = np.empty((T, n, N), dtype=np.int32)
    logits = np.empty((T, n, N, N_ACTIONS), dtype=np.float64)
    rc = lib().orc_evaluate(C.byref(cfg), C.c_uint64(seed), _ptr(p), int(emulate_bf16), n, _ptr(env_ids), T,
                            t_global0, st, _ptr(fa), int(greedy), _ptr(ep), _ptr(rs), _ptr(ls), _ptr(actions),
                            _ptr(logits))
    if rc != 0:
        raise ValueError("orc_evaluate rejected its arguments")
    return Evaluation(ep, rs, ls, actions, logits, list(st))


def gae(values, rewards, dones, gamma: float, lam: float):
    """values [T+1][E][N], rewards [T][E][N], dones [T][E] -> (adv, ret) float64."""
    v = np.ascontiguousarray(values, dtype=np.float32)
    r = np.ascontiguousarray(rewards, dtype=np.float32)
    d = np.ascontiguousarray(dones, dtype=np.uint8)
    T, E, N = r.shape
    assert v.shape == (T + 1, E, N) and d.shape == (T, E)
    adv = np.empty((T, E, N), dtype=np.float64)
    ret = np.empty((T, E, N), dtype=np.float64)
    lib().orc_gae(T, E, N, _ptr(v), _ptr(r), _ptr(d), gamma, lam, _ptr(adv), _ptr(ret))
    return adv, ret


def gae_bruteforce(values, rewards, dones, gamma: float, lam: float):
    v = np.ascontiguousarray(values, dtype=np.float32)
    r = np.ascontiguousarray(rewards, dtype=np.float32)
    d = np.ascontiguousarray(dones, dtype=np.uint8)
    T, E, N = r.shape
    adv = np.empty((T, E, N), dtype=np.float64)
    lib().orc_gae_bruteforce(T, E, N, _ptr(v), _ptr(r), _ptr(d), gamma, lam, _ptr(adv))
    return adv
