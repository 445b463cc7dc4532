"""GPU parity tests: the CUDA library (through its C ABI) against the CPU oracle."""
import numpy as np
import pytest

import oracle
from paper_2107_01460_b200 import binding, workloads as wl

from parity import check_against_oracle, run_gpu

pytestmark = pytest.mark.gpu

FP32 = binding.MAVA_PRECISION_FP32
BF16 = binding.MAVA_PRECISION_BF16


def _precision(w):
    return BF16 if w["precision"] == "bf16" else FP32


def _tc_available(w):
    import ctypes as C

    cfg = binding.make_config(w, precision=BF16)
    return bool(binding.lib().mava_params_count(C.byref(cfg))) and _try_create(cfg)


def _try_create(cfg):
    try:
        cfg2 = binding.mava_config_t.from_buffer_copy(cfg)
        cfg2.n_envs, cfg2.max_T = 4, 2
        binding.Rollout(cfg2).close()
        return True
    except binding.MavaError as e:
        if e.code == binding.MAVA_ERR_UNSUPPORTED:
            return False
        raise


# ---- whole small config, every environment checked -------------------------------------------

@pytest.mark.parametrize("bias_scale", [0.0, 0.5])
def test_cfg0_fp32_every_row(bias_scale):
    w = wl.workload(0)
    params = wl.make_params(w, bias_scale=bias_scale)
    ro, _ = run_gpu(w, FP32, w["T"], params=params)
    out = check_against_oracle(w, ro, params, w["T"], FP32, np.arange(w["n_envs"]))
    print(out)


def test_cfg0_longer_than_the_cap_crosses_resets():
    w = wl.workload(0)
    params = wl.make_params(w)
    T = 120
    ro, _ = run_gpu(w, FP32, T, params=params)
    assert int(ro.dones.sum()) >= 2 * w["n_envs"]
    check_against_oracle(w, ro, params, T, FP32, np.arange(w["n_envs"]))


# ---- reduced versions of the larger configs (several tiles and a ragged last tile) -----------

@pytest.mark.parametrize("idx,n_envs,T", [(1, 77, 60), (2, 101, 110), (3, 45, 105), (4, 37, 40)])
def test_reduced_configs_fp32(idx, n_envs, T):
    w = wl.workload(idx)
    params = wl.make_params(w, bias_scale=0.1)
    ro, _ = run_gpu(w, FP32, T, n_envs=n_envs, params=params)
    ids = wl.sample_env_ids(n_envs, 6, 6, 6, seed=idx)
    out = check_against_oracle(w, ro, params, T, FP32, ids)
    print(idx, out)


@pytest.mark.parametrize("idx,n_envs,T,mode", [(1, 333, 60, ""), (2, 300, 110, ""), (3, 200, 105, ""),
                                               (4, 150, 40, ""), (0, 16, 32, "tmem"), (1, 333, 60, "tmem"),
                                               (2, 300, 110, "tmem"), (1, 333, 60, "wide"), (2, 300, 110, "wide"),
                                               (1, 1500, 40, ""), (2, 1000, 40, ""), (1, 1500, 40, "wide"),
                                               # H = 256 with more tiles than one round holds and an odd count: a second
                                               # round in which one thread group of a CTA has no tile (on 148 SMs)
                                               (4, 4737, 12, ""), (3, 9473, 7, "")])
def test_reduced_configs_bf16(idx, n_envs, T, mode):
    """mode "tmem" keeps the hidden activations in tensor memory (the layout H = 256 always uses);
    "wide" forces 128-row tiles where the batch is small enough for the few-rows form of the kernel
    (H = 128: up to 16 rows per SM at 333 / 300 environments, up to 32 at 1500 / 1000)."""
    w = wl.workload(idx)
    if not _tc_available(w):
        pytest.skip("bf16 tensor-core path not compiled for this shape")
    params = wl.make_params(w, bias_scale=0.1)
    flags = binding.MAVA_FLAG_WRITE_LOGITS | {"": 0, "tmem": binding.MAVA_FLAG_HIDDEN_IN_TMEM,
                                              "wide": binding.MAVA_FLAG_WIDE_TILES}[mode]
    ro, _ = run_gpu(w, BF16, T, n_envs=n_envs, params=params, flags=flags)
    ids = wl.sample_env_ids(n_envs, 6, 6, 6, seed=idx)
    out = check_against_oracle(w, ro, params, T, BF16, ids)
    print(idx, out)


@pytest.mark.parametrize("idx,n_envs", [(1, 1024), (1, 2000), (2, 700), (2, 1400)])
def test_few_rows_form_equals_wide_tiles(idx, n_envs):
    """The few-rows form of the bf16 kernel (rows as the N operand of the MMA) forms the same products
    in the same order as the 128-row form: every output is bit-identical."""
    w = wl.workload(idx)
    T = 48
    params = wl.make_params(w, bias_scale=0.1)
    outs = []
    for extra in (0, binding.MAVA_FLAG_WIDE_TILES):
        ro, _ = run_gpu(w, BF16, T, n_envs=n_envs, params=params, flags=binding.MAVA_FLAG_WRITE_LOGITS | extra)
        outs.append({k: getattr(ro, k)[:T + (1 if k == "values" else 0)].cpu().numpy().copy()
                     for k in ("obs", "actions", "logp", "values", "rewards", "dones", "logits", "adv", "ret")})
    for k in outs[0]:
        assert np.array_equal(outs[0][k].view(np.uint8), outs[1][k].view(np.uint8)), k


# ---- full-size configs in the launch configuration the benchmark times ------------------------

@pytest.mark.parametrize("idx", [0, 1, 2, 3, 4])
def test_full_size_configs(idx):
    """Every workload at its full size, in bf16 with default flags (the launch shape the benchmark times).  Environment
    arrays: all environments.  Network, sampler and log-probabilities: the first 64, the last 64 and 128 seeded-random
    environments at every step, against the float64 oracle (2e-2) and against the oracle with bf16-rounded operands
    (2e-3, which also sets the margin of the action rule)."""
    w = wl.workload(idx)
    precision = _precision(w) if _tc_available(w) else FP32
    params = wl.make_params(w)
    T, E = w["T"], w["n_envs"]
    ro, _ = run_gpu(w, precision, T, params=params)
    ids = wl.sample_env_ids(E, 64, 64, 128, seed=idx)
    out = check_against_oracle(w, ro, params, T, precision, ids, obs_env_ids=None if E <= 256 else ids)
    print(idx, precision, len(ids), out)


# ---- hand-worked transitions through set_state + forced actions -------------------------------

def test_hand_worked_steps_on_the_gpu():
    import torch

    w = wl.workload(0)
    cfg = binding.make_config(w, precision=FP32, max_T=1, n_envs=6)
    ro = binding.Rollout(cfg)
    params = torch.from_numpy(wl.make_params(w)).cuda()
    far = [7, 7, 1, 7, 0, 1]
    # record: a0(r,c,l) a1(r,c,l) f0(r,c,l) f1(r,c,l) step episode total
    states = np.array([
        [2, 2, 1, 2, 4, 1, *far, 0, 0, 2],             # head-on to the same cell
        [2, 2, 1, 2, 3, 1, *far, 0, 0, 2],             # follow into a vacated cell
        [0, 5, 1, 5, 5, 1, *far, 0, 0, 2],             # wall
        [3, 2, 1, 2, 3, 2, 3, 3, 3, 6, 6, 2, 0, 0, 5],  # joint load collects level 3 of 5
        [3, 2, 1, 2, 3, 1, 3, 3, 1, 6, 6, 2, 0, 0, 3],  # collected food still blocks this step
        [3, 2, 1, 6, 6, 1, *far, 49, 0, 2],            # cap
    ], dtype=np.int32)
    acts = np.array([[4, 3], [4, 4], [1, 0], [5, 5], [5, 2], [0, 0]], dtype=np.int32)[None]
    ro.set_state(states)
    ro.run_forced(params, 1, torch.from_numpy(acts).cuda())
    assert ro.status() == 0
    after = ro.get_state()
    assert after[0, :6].tolist() == [2, 2, 1, 2, 4, 1]
    assert after[1, :6].tolist() == [2, 2, 1, 2, 4, 1]
    assert after[2, :3].tolist() == [0, 5, 1]
    assert after[3, 8] == 0 and after[3, 11] == 2
    assert after[4, 8] == 0 and after[4, 3:5].tolist() == [2, 3]
    rew = ro.rewards[0].cpu().numpy()
    assert rew[3].tolist() == [np.float32(3) / np.float32(5)] * 2
    assert rew[4].tolist() == [np.float32(1) / np.float32(3)] * 2
    assert ro.dones[0].cpu().numpy().tolist() == [0, 0, 0, 0, 0, 1]
    assert after[5, 12:14].tolist() == [0, 1]  # fresh episode 1
    fresh = oracle.env_reset(oracle.make_config(w), w["seed"], 5, 1)
    assert after[5, :2].tolist() == [fresh.agent_r[0], fresh.agent_c[0]]


# ---- determinism, continuation, reset ------------------------------------------------------------

def test_two_runs_give_identical_bytes_and_reset_replays():
    import torch

    w = wl.workload(2)
    T = 50
    cfg = binding.make_config(w, precision=FP32, max_T=T, n_envs=95)
    ro = binding.Rollout(cfg)
    params = torch.from_numpy(wl.make_params(w)).cuda()
    ro.run(params, T)
    first = [t.clone() for t in (ro.obs, ro.actions, ro.logp, ro.values, ro.rewards, ro.dones)]
    ro.reset(w["seed"])
    ro.run(params, T)
    for a, b in zip(first, (ro.obs, ro.actions, ro.logp, ro.values, ro.rewards, ro.dones)):
        assert torch.equal(a, b)
    assert ro.status() == 0


def test_two_calls_continue_like_one():
    import torch

    w = wl.workload(1)
    cfg = binding.make_config(w, precision=FP32, max_T=70, n_envs=40)
    params = torch.from_numpy(wl.make_params(w)).cuda()
    a = binding.Rollout(cfg)
    a.run(params, 70)
    b = binding.Rollout(cfg)
    b.run(params, 30)
    obs1, act1 = b.obs[:30].clone(), b.actions[:30].clone()
    b.run(params, 40)
    assert torch.equal(a.obs[:30], obs1) and torch.equal(a.actions[:30], act1)
    assert torch.equal(a.obs[30:70], b.obs[:40]) and torch.equal(a.actions[30:70], b.actions[:40])
    assert torch.equal(a.values[70], b.values[40])
    assert np.array_equal(a.get_state(), b.get_state())


def test_capacity_and_argument_errors():
    import torch

    w = wl.workload(0)
    cfg = binding.make_config(w, precision=FP32, max_T=8)
    ro = binding.Rollout(cfg, with_gae=False)
    params = torch.from_numpy(wl.make_params(w)).cuda()
    with pytest.raises(binding.MavaError) as e:
        ro.run(params, 9)
    assert e.value.code == binding.MAVA_ERR_CAPACITY
    with pytest.raises(binding.MavaError) as e:
        ro.gae(0.99, 0.95)  # no run yet and no adv/ret buffers
    assert e.value.code == binding.MAVA_ERR_INVALID_ARG
    ro.run(params, 8)
    assert ro.status() == 0 and ro.launch_count() >= 3


# ---- GAE on arbitrary data, odd shapes ------------------------------------------------------------

@pytest.mark.parametrize("idx,n_envs,T", [(0, 16, 1), (0, 5, 13), (2, 47, 37), (4, 33, 64), (1, 300, 128), (3, 9, 250),
                                              (4, 2100, 37), (2, 5464, 100),  # these two take the float4 variant
                                              # the copy-engine variant (E a multiple of 16): environments that straddle
                                              # a thread's four columns and a ragged last tile, single-step last chunk,
                                              # two agents and more chunks than a warp has lanes, a long T
                                              (2, 5488, 101), (4, 2112, 37), (1, 8208, 130), (0, 8192, 200),
                                              (0, 8192, 255)])  # too long for three stages: back to the plain scan
def test_gae_on_random_trajectories(idx, n_envs, T):
    import torch

    w = wl.workload(idx)
    cfg = binding.make_config(w, precision=FP32, max_T=T, n_envs=n_envs)
    ro = binding.Rollout(cfg)
    ro.run(torch.from_numpy(wl.make_params(w)).cuda(), T)
    g = torch.Generator(device="cuda").manual_seed(idx)
    ro.values.copy_(torch.randn(ro.values.shape, generator=g, device="cuda"))
    ro.rewards.copy_(torch.rand(ro.rewards.shape, generator=g, device="cuda"))
    ro.dones.copy_((torch.rand(ro.dones.shape, generator=g, device="cuda") < 0.1).to(torch.uint8))
    for gamma, lam in [(0.99, 0.95), (1.0, 1.0), (0.9, 0.0)]:
        ro.gae(gamma, lam)
        adv, ret = oracle.gae(ro.values.cpu().numpy(), ro.rewards.cpu().numpy(), ro.dones.cpu().numpy(),
                              float(np.float32(gamma)), float(np.float32(lam)))
        ga, gr = ro.adv.cpu().numpy(), ro.ret.cpu().numpy()
        assert np.max(np.abs(ga - adv) / np.maximum(1, np.abs(adv))) <= 1e-5
        assert np.max(np.abs(gr - ret) / np.maximum(1, np.abs(ret))) <= 1e-5


# ---- tensor-core path: determinism, continuation, sharding, forcing, degenerate sizes ----------

@pytest.mark.parametrize("idx,n_envs", [(1, 150), (4, 50), (3, 40)])
def test_bf16_two_calls_continue_like_one_and_runs_repeat(idx, n_envs):
    import torch

    w = wl.workload(idx)
    cfg = binding.make_config(w, precision=BF16, max_T=50, n_envs=n_envs)
    params = torch.from_numpy(wl.make_params(w, bias_scale=0.1)).cuda()
    a = binding.Rollout(cfg)
    a.run(params, 50)
    whole = [t.clone() for t in (a.obs, a.actions, a.logp, a.values, a.rewards, a.dones)]
    a.reset(w["seed"])
    a.run(params, 50)
    for x, y in zip(whole, (a.obs, a.actions, a.logp, a.values, a.rewards, a.dones)):
        assert torch.equal(x, y)  # same seed, same bytes
    b = binding.Rollout(cfg)
    b.run(params, 20)
    first = [t[:20].clone() for t in (b.obs, b.actions, b.logp, b.rewards, b.dones)]
    b.run(params, 30)
    for x, y, z in zip(first, (b.obs, b.actions, b.logp, b.rewards, b.dones), (a.obs, a.actions, a.logp, a.rewards, a.dones)):
        assert torch.equal(z[:20], x) and torch.equal(z[20:50], y[:30])
    assert torch.equal(a.values[50], b.values[30]) and np.array_equal(a.get_state(), b.get_state())
    assert a.status() == 0 and b.status() == 0


@pytest.mark.parametrize("idx", [2, 4])
def test_env_shards_reproduce_the_whole_batch_on_the_gpu(idx):
    """Two handles with first_env offsets give the bytes of one handle over all environments."""
    import torch

    w = wl.workload(idx)
    T, n = 30, 90
    params = torch.from_numpy(wl.make_params(w)).cuda()
    whole = binding.Rollout(binding.make_config(w, precision=BF16, max_T=T, n_envs=n))
    whole.run(params, T)
    cut = 37
    lo = binding.Rollout(binding.make_config(w, precision=BF16, max_T=T, n_envs=cut))
    hi = binding.Rollout(binding.make_config(w, precision=BF16, max_T=T, n_envs=n - cut, first_env=cut))
    lo.run(params, T)
    hi.run(params, T)
    for name in ("obs", "actions", "rewards", "dones", "logp", "values"):
        full = getattr(whole, name)
        assert torch.equal(full[:, :cut], getattr(lo, name)) and torch.equal(full[:, cut:], getattr(hi, name)), name


@pytest.mark.parametrize("precision", [FP32, BF16])
@pytest.mark.parametrize("idx,n_envs,T", [(0, 1, 1), (2, 1, 3), (4, 1, 2), (3, 2, 1)])
def test_degenerate_sizes(idx, n_envs, T, precision):
    w = wl.workload(idx)
    params = wl.make_params(w)
    ro, _ = run_gpu(w, precision, T, n_envs=n_envs, params=params)
    check_against_oracle(w, ro, params, T, precision, np.arange(n_envs))


def test_forced_actions_on_the_tensor_path():
    """Teacher forcing in bf16: the oracle's own free-running actions, replayed on the GPU."""
    import torch

    w = wl.workload(1)
    T, n = 40, 70
    params = wl.make_params(w)
    ocfg = oracle.make_config(w)
    free = oracle.rollout(ocfg, w["seed"], params, T, np.arange(n))
    cfg = binding.make_config(w, precision=BF16, max_T=T, n_envs=n)
    ro = binding.Rollout(cfg)
    ro.run_forced(torch.from_numpy(params).cuda(), T, torch.from_numpy(free.actions).cuda())
    assert ro.status() == 0
    assert np.array_equal(ro.actions.cpu().numpy(), free.actions)
    assert np.array_equal(ro.obs.cpu().numpy().view(np.uint32), free.obs.view(np.uint32))
    assert np.array_equal(ro.rewards.cpu().numpy(), free.rewards) and np.array_equal(ro.dones.cpu().numpy(), free.dones)
    lp = ro.logp.cpu().numpy()
    assert np.all(np.abs(lp - free.logp) <= 2e-2 * (1 + np.abs(free.logp)))


@pytest.mark.parametrize("idx,n_envs,T", [(1, 200, 41), (2, 900, 64), (3, 60, 33), (0, 16, 5), (4, 80, 24)])
def test_collect_host_delivers_the_bytes_of_run_and_gae(idx, n_envs, T):
    """The host-buffer call (parameters in, whole trajectory out, rolled out in pieces whose copies
    overlap the kernels) against run + gae on a second handle: every array bit for bit, twice in a row."""
    import torch

    w = wl.workload(idx)
    flags = binding.MAVA_FLAG_WRITE_LOGITS
    params = torch.from_numpy(wl.make_params(w, bias_scale=0.1))
    a = binding.Rollout(binding.make_config(w, precision=BF16, max_T=T, n_envs=n_envs, flags=flags))
    b = binding.Rollout(binding.make_config(w, precision=BF16, max_T=T, n_envs=n_envs, flags=flags))
    names = ("obs", "actions", "logp", "values", "rewards", "dones", "adv", "ret", "logits")
    out = {n: torch.empty_like(getattr(b, n), device="cpu").pin_memory() for n in names}
    p_dev = params.cuda()
    for _ in range(2):
        a.run(p_dev, T)
        a.gae(wl.GAMMA, wl.LAMBDA)
        b.collect_host(params.pin_memory(), T, wl.GAMMA, wl.LAMBDA, out)
        for n in names:
            rows = T + 1 if n == "values" else T
            assert torch.equal(out[n][:rows], getattr(a, n)[:rows].cpu()), n
    assert np.array_equal(a.get_state(), b.get_state())
    assert a.status() == 0 and b.status() == 0
