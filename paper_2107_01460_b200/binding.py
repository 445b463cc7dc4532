"""Thin ctypes binding of libmava_rollout.so: same entry-point names as the C header, argument
marshalling only.  PyTorch is used for device memory and streams; every step of the rollout and
of GAE runs inside the library's CUDA kernels.  There is no fallback: if the shared library has
not been built (``python -m paper_2107_01460_b200.build``) loading raises."""
from __future__ import annotations

import ctypes as C
import os

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmava_rollout.so")

MAVA_OK = 0
MAVA_ERR_INVALID_ARG = -1
MAVA_ERR_UNSUPPORTED = -2
MAVA_ERR_CUDA = -3
MAVA_ERR_DEVICE_TIMEOUT = -4
MAVA_ERR_CAPACITY = -5
MAVA_NET_SHARED_TORSO = 0
MAVA_NET_CENTRAL_CRITIC = 1
MAVA_NET_RECURRENT = 2
MAVA_PRECISION_FP32 = 0
MAVA_PRECISION_BF16 = 1
MAVA_FLAG_WRITE_LOGITS = 1
MAVA_FLAG_HIDDEN_IN_TMEM = 2
MAVA_FLAG_WIDE_TILES = 4
MAVA_FLAG_UPDATE_FP32 = 8
MAVA_EXPIRE_GAE = 1
MAVA_EXPIRE_ROLLOUT = 2
MAVA_GAE_MAX_T = 1024
N_ACTIONS = 6

EXPORTS = [
    "mava_params_count", "mava_rollout_create", "mava_rollout_run", "mava_rollout_run_forced", "mava_gae",
    "mava_rollout_reset", "mava_rollout_status", "mava_state_record_len", "mava_rollout_get_state",
    "mava_rollout_set_state", "mava_rollout_collect_host", "mava_rollout_launch_count", "mava_rollout_destroy",
    "mava_strerror", "mava_rollout_run_static", "mava_rollout_evaluate", "mava_ppo_defaults", "mava_ppo_grad",
    "mava_adam_step", "mava_ppo_grad_envs", "mava_debug_expire_next_wait", "mava_rollout_get_hidden", "mava_ppo_update",
]


class mava_ppo_hyper_t(C.Structure):
    _fields_ = [(n, C.c_float) for n in ("clip_eps", "ent_coef", "vf_coef", "lr", "beta1", "beta2", "adam_eps", "max_grad_norm")]


class mava_config_t(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "grid", "n_agents", "n_food", "max_agent_level", "view_radius", "episode_cap", "n_envs", "max_T", "hidden",
        "net_kind", "precision", "flags", "first_env", "env_kind")] + [("seed", C.c_uint64)]


class mava_buffers_t(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "obs", "actions", "logp", "values", "rewards", "dones", "adv", "ret", "logits")]


class MavaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


_lib = None


def lib():
    """The loaded shared library (raises FileNotFoundError / OSError if it was not built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2107_01460_b200.build` (there is no fallback)")
        L = C.CDLL(LIB_PATH)
        cfgp, bufp, vp = C.POINTER(mava_config_t), C.POINTER(mava_buffers_t), C.c_void_p
        L.mava_params_count.argtypes = [cfgp]; L.mava_params_count.restype = C.c_size_t
        L.mava_state_record_len.argtypes = [cfgp]; L.mava_state_record_len.restype = C.c_int32
        L.mava_rollout_create.argtypes = [cfgp, bufp, vp, C.POINTER(vp)]; L.mava_rollout_create.restype = C.c_int
        L.mava_rollout_run.argtypes = [vp, vp, C.c_int32]; L.mava_rollout_run.restype = C.c_int
        L.mava_rollout_run_forced.argtypes = [vp, vp, C.c_int32, vp]; L.mava_rollout_run_forced.restype = C.c_int
        L.mava_rollout_evaluate.argtypes = [vp, vp, C.c_int32, C.c_int32, vp, vp, vp, vp]
        L.mava_rollout_evaluate.restype = C.c_int
        L.mava_gae.argtypes = [vp, C.c_float, C.c_float]; L.mava_gae.restype = C.c_int
        L.mava_rollout_reset.argtypes = [vp, C.c_uint64]; L.mava_rollout_reset.restype = C.c_int
        L.mava_rollout_status.argtypes = [vp]; L.mava_rollout_status.restype = C.c_int
        L.mava_rollout_get_state.argtypes = [vp, vp]; L.mava_rollout_get_state.restype = C.c_int
        L.mava_rollout_set_state.argtypes = [vp, vp]; L.mava_rollout_set_state.restype = C.c_int
        L.mava_rollout_collect_host.argtypes = [vp, vp, C.c_int32, C.c_float, C.c_float, bufp]
        L.mava_rollout_collect_host.restype = C.c_int
        L.mava_rollout_launch_count.argtypes = [vp]; L.mava_rollout_launch_count.restype = C.c_int64
        L.mava_rollout_destroy.argtypes = [vp]; L.mava_rollout_destroy.restype = None
        L.mava_strerror.argtypes = [C.c_int]; L.mava_strerror.restype = C.c_char_p
        L.mava_rollout_run_static.argtypes = [cfgp, bufp, vp, C.c_int32, vp]
        L.mava_rollout_run_static.restype = C.c_int
        hpp = C.POINTER(mava_ppo_hyper_t)
        L.mava_ppo_defaults.argtypes = [hpp]; L.mava_ppo_defaults.restype = None
        L.mava_ppo_grad.argtypes = [vp, vp, hpp, vp, vp]; L.mava_ppo_grad.restype = C.c_int
        L.mava_ppo_grad_envs.argtypes = [vp, vp, hpp, vp, C.c_int32, vp, vp]; L.mava_ppo_grad_envs.restype = C.c_int
        L.mava_adam_step.argtypes = [vp, vp, vp, vp, vp, C.c_int32, hpp]; L.mava_adam_step.restype = C.c_int
        L.mava_ppo_update.argtypes = [vp, vp, vp, vp, vp, hpp, C.c_int32, C.c_int32, vp, C.c_int32, vp]
        L.mava_ppo_update.restype = C.c_int
        L.mava_rollout_get_hidden.argtypes = [vp, vp]; L.mava_rollout_get_hidden.restype = C.c_int
        L.mava_debug_expire_next_wait.argtypes = [vp, C.c_int32]; L.mava_debug_expire_next_wait.restype = C.c_int
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().mava_strerror(code).decode()


def make_config(w: dict, precision: int | None = None, flags: int = 0, max_T: int | None = None,
                n_envs: int | None = None, seed: int | None = None, first_env: int = 0) -> mava_config_t:
    """mava_config_t from a workload description (see ``workloads.WORKLOADS``)."""
    if precision is None:
        precision = MAVA_PRECISION_BF16 if w.get("precision") == "bf16" else MAVA_PRECISION_FP32
    return mava_config_t(
        grid=w["grid"], n_agents=w["n_agents"], n_food=w["n_food"], max_agent_level=w["max_agent_level"],
        view_radius=w["view_radius"], episode_cap=w["episode_cap"], n_envs=w["n_envs"] if n_envs is None else n_envs,
        max_T=w["T"] if max_T is None else max_T, hidden=w["hidden"], net_kind=w["net_kind"], precision=precision,
        flags=flags, first_env=first_env, env_kind=w.get("env_kind", 0), seed=w["seed"] if seed is None else seed)


def update_on_tensor_cores(cfg: mava_config_t) -> bool:
    """Whether mava_ppo_grad takes the bf16 tensor-core kernels for a handle of this configuration: the shared-torso
    shapes with H <= 128 and D <= 80 (one fused kernel), and H = 256 with 64 < D <= 96 (row kernel + weight kernel; with
    a centralised critic both nets)."""
    if cfg.precision != MAVA_PRECISION_BF16 or cfg.flags & MAVA_FLAG_UPDATE_FP32:
        return False
    D = 77 + cfg.n_agents
    return (cfg.net_kind == MAVA_NET_SHARED_TORSO and cfg.hidden <= 128 and D <= 80) or (cfg.hidden == 256 and 64 < D <= 96)


def ppo_defaults() -> mava_ppo_hyper_t:
    hp = mava_ppo_hyper_t()
    lib().mava_ppo_defaults(C.byref(hp))
    return hp


def _check(code: int, where: str):
    if code != MAVA_OK:
        raise MavaError(code, where)


def mava_rollout_run_static(cfg: mava_config_t, buffers: mava_buffers_t, params_dev_ptr: int, T: int,
                            cuda_stream: int | None = None) -> int:
    """The allocation-free rollout for callers that must not allocate device memory (see the
    header): returns the C status code; `buffers` holds raw device pointers the caller owns."""
    return int(lib().mava_rollout_run_static(C.byref(cfg), C.byref(buffers), params_dev_ptr, T, cuda_stream))


class Rollout:
    """Owns the torch device tensors of one handle and forwards to the C entry points."""

    def __init__(self, cfg: mava_config_t, device="cuda:0", stream=None, with_gae: bool = True):
        import torch

        self.torch = torch
        self.cfg = cfg
        self.device = torch.device(device)
        E, N, T = cfg.n_envs, cfg.n_agents, cfg.max_T
        self.D = 77 + N
        self.n_params = int(lib().mava_params_count(C.byref(cfg)))
        if self.n_params == 0:
            raise MavaError(MAVA_ERR_INVALID_ARG, "mava_params_count")
        dev = self.device
        f32, i32, u8 = torch.float32, torch.int32, torch.uint8
        self.obs = torch.empty((T, E, N, self.D), dtype=f32, device=dev)
        self.actions = torch.empty((T, E, N), dtype=i32, device=dev)
        self.logp = torch.empty((T, E, N), dtype=f32, device=dev)
        self.values = torch.empty((T + 1, E, N), dtype=f32, device=dev)
        self.rewards = torch.empty((T, E, N), dtype=f32, device=dev)
        self.dones = torch.empty((T, E), dtype=u8, device=dev)
        self.adv = torch.empty((T, E, N), dtype=f32, device=dev) if with_gae else None
        self.ret = torch.empty((T, E, N), dtype=f32, device=dev) if with_gae else None
        self.logits = (torch.empty((T, E, N, N_ACTIONS), dtype=f32, device=dev)
                       if cfg.flags & MAVA_FLAG_WRITE_LOGITS else None)
        ptr = lambda t: None if t is None else t.data_ptr()  # noqa: E731
        self.buffers = mava_buffers_t(ptr(self.obs), ptr(self.actions), ptr(self.logp), ptr(self.values),
                                      ptr(self.rewards), ptr(self.dones), ptr(self.adv), ptr(self.ret),
                                      ptr(self.logits))
        self.stream = stream if stream is not None else torch.cuda.current_stream(dev)
        self.handle = C.c_void_p()
        with torch.cuda.device(dev):
            _check(lib().mava_rollout_create(C.byref(cfg), C.byref(self.buffers), C.c_void_p(self.stream.cuda_stream),
                                             C.byref(self.handle)), "mava_rollout_create")

    # -- one method per C entry point ---------------------------------------------------------
    def run(self, params, T: int):
        assert params.is_cuda and params.dtype == self.torch.float32 and params.numel() == self.n_params
        _check(lib().mava_rollout_run(self.handle, params.data_ptr(), T), "mava_rollout_run")

    def run_forced(self, params, T: int, actions):
        assert actions.is_cuda and actions.dtype == self.torch.int32 and actions.is_contiguous()
        assert params.is_cuda and params.numel() == self.n_params
        _check(lib().mava_rollout_run_forced(self.handle, params.data_ptr(), T, actions.data_ptr()),
               "mava_rollout_run_forced")

    def evaluate(self, params, T: int, greedy: bool = True, want_actions: bool = False):
        """An evaluation block of T steps (mava_rollout_evaluate): returns device tensors
        (ep_count [E] int32, ret_sum [E] float32, len_sum [E] int32, actions [T][E][N] int32 or None)."""
        t = self.torch
        assert params.is_cuda and params.dtype == t.float32 and params.numel() == self.n_params
        E, N = self.cfg.n_envs, self.cfg.n_agents
        dev = params.device
        ep_count = t.empty(E, dtype=t.int32, device=dev)
        ret_sum = t.empty(E, dtype=t.float32, device=dev)
        len_sum = t.empty(E, dtype=t.int32, device=dev)
        actions = t.empty((T, E, N), dtype=t.int32, device=dev) if want_actions else None
        _check(lib().mava_rollout_evaluate(self.handle, params.data_ptr(), T, int(greedy), ep_count.data_ptr(),
                                           ret_sum.data_ptr(), len_sum.data_ptr(),
                                           actions.data_ptr() if want_actions else None), "mava_rollout_evaluate")
        return ep_count, ret_sum, len_sum, actions

    def gae(self, gamma: float, lam: float):
        _check(lib().mava_gae(self.handle, gamma, lam), "mava_gae")

    def ppo_grad(self, params, hp: "mava_ppo_hyper_t | None" = None, env_ids=None):
        """Loss terms [4] (total, actor, entropy, value) and dL/dparams of the last run's rows (of the environments
        `env_ids`, an int32 device tensor, when given); device tensors."""
        import torch

        hp = ppo_defaults() if hp is None else hp
        grad = torch.empty_like(params)
        terms = torch.empty(4, dtype=torch.float32, device=params.device)
        if env_ids is not None:
            assert env_ids.is_cuda and env_ids.dtype == torch.int32 and env_ids.is_contiguous()
            _check(lib().mava_ppo_grad_envs(self.handle, params.data_ptr(), C.byref(hp), env_ids.data_ptr(), env_ids.numel(),
                                            grad.data_ptr(), terms.data_ptr()), "mava_ppo_grad_envs")
            return terms, grad
        _check(lib().mava_ppo_grad(self.handle, params.data_ptr(), C.byref(hp), grad.data_ptr(), terms.data_ptr()), "mava_ppo_grad")
        return terms, grad

    def adam_step(self, params, grad, m, v, step: int, hp: "mava_ppo_hyper_t | None" = None):
        """One clipped Adam step on `params` in place (m, v: the caller's moment tensors, zero at first)."""
        hp = ppo_defaults() if hp is None else hp
        _check(lib().mava_adam_step(self.handle, params.data_ptr(), grad.data_ptr(), m.data_ptr(), v.data_ptr(), step,
                                    C.byref(hp)), "mava_adam_step")

    def ppo_update(self, params, m, v, perm, minibatches: int, first_step: int, hp: "mava_ppo_hyper_t | None" = None):
        """`perm.shape[0]` passes of `minibatches` minibatches each over the last run's rows (mava_ppo_update): params, m,
        v change in place; returns the loss terms [passes * minibatches][4] (device tensor)."""
        import torch

        hp = ppo_defaults() if hp is None else hp
        assert perm.is_cuda and perm.dtype == torch.int32 and perm.is_contiguous() and perm.shape[1] == self.cfg.n_envs
        grad = torch.empty_like(params)
        terms = torch.empty((perm.shape[0] * minibatches, 4), dtype=torch.float32, device=params.device)
        _check(lib().mava_ppo_update(self.handle, params.data_ptr(), m.data_ptr(), v.data_ptr(), grad.data_ptr(), C.byref(hp),
                                     perm.shape[0], minibatches, perm.data_ptr(), first_step, terms.data_ptr()), "mava_ppo_update")
        return terms

    def reset(self, seed: int):
        _check(lib().mava_rollout_reset(self.handle, seed), "mava_rollout_reset")

    def status(self) -> int:
        return int(lib().mava_rollout_status(self.handle))

    def debug_expire_next_wait(self, which: int):
        _check(lib().mava_debug_expire_next_wait(self.handle, which), "mava_debug_expire_next_wait")

    def launch_count(self) -> int:
        return int(lib().mava_rollout_launch_count(self.handle))

    def get_state(self):
        import numpy as np

        n = int(lib().mava_state_record_len(C.byref(self.cfg)))
        out = np.empty((self.cfg.n_envs, n), dtype=np.int32)
        _check(lib().mava_rollout_get_state(self.handle, out.ctypes.data), "mava_rollout_get_state")
        return out

    def get_hidden(self):
        """Recurrent policy: the hidden vectors the next run starts from, [E][N][H] float32 (numpy)."""
        import numpy as np

        out = np.empty((self.cfg.n_envs, self.cfg.n_agents, self.cfg.hidden), dtype=np.float32)
        _check(lib().mava_rollout_get_hidden(self.handle, out.ctypes.data), "mava_rollout_get_hidden")
        return out

    def set_state(self, records):
        import numpy as np

        rec = np.ascontiguousarray(records, dtype=np.int32)
        assert rec.shape == (self.cfg.n_envs, int(lib().mava_state_record_len(C.byref(self.cfg))))
        _check(lib().mava_rollout_set_state(self.handle, rec.ctypes.data), "mava_rollout_set_state")

    def collect_host(self, params_host, T: int, gamma: float, lam: float, out: dict):
        """`out`: dict name -> pinned CPU tensor (any subset of the buffer names)."""
        hb = mava_buffers_t(*[(out[n].data_ptr() if n in out else None) for n, _ in mava_buffers_t._fields_])
        _check(lib().mava_rollout_collect_host(self.handle, params_host.data_ptr(), T, gamma, lam, C.byref(hb)),
               "mava_rollout_collect_host")

    def close(self):
        if self.handle:
            lib().mava_rollout_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
