"""Warehouse workload family on the GPU (through the C ABI) against the oracle: the same comparison as for the foraging
workloads -- environment arrays and final states bit for bit under the GPU's own actions, network outputs within the
path's tolerance, sampler exactly -- plus hand-worked transitions forced on the GPU."""
import numpy as np
import pytest

import oracle
from paper_2107_01460_b200 import binding, workloads as wl

from parity import check_against_oracle, run_gpu

pytestmark = pytest.mark.gpu
FP32, BF16 = binding.MAVA_PRECISION_FP32, binding.MAVA_PRECISION_BF16
WH0, WH1, WH2 = "wh0_tiny_8x8_2r2s_h64", "wh1_10x10_3r3s_h128", "wh2_10x10_3r3s_h128_collisions_end"


@pytest.mark.parametrize("precision", [FP32, BF16])
@pytest.mark.parametrize("name,n_envs,T", [(WH0, 16, 120), (WH1, 101, 110), (WH2, 300, 60), (WH2, 1, 5)])
def test_warehouse_rollout(name, n_envs, T, precision):
    w = wl.workload(name)
    params = wl.make_params(w, bias_scale=0.1)
    ro, _ = run_gpu(w, precision, T, n_envs=n_envs, params=params)
    ids = wl.sample_env_ids(n_envs, 8, 8, 8, seed=3)
    out = check_against_oracle(w, ro, params, T, precision, ids)
    if name == WH2 and n_envs > 1:
        assert int(ro.dones[:T].sum()) > n_envs  # robot conflicts end episodes long before the cap
    print(name, precision, out)
    ro.close()


@pytest.mark.parametrize("name", [WH1, WH2])
def test_warehouse_full_size(name):
    w = wl.workload(name)
    params = wl.make_params(w)
    ro, _ = run_gpu(w, BF16, w["T"], params=params)
    ids = wl.sample_env_ids(w["n_envs"], 64, 64, 128, seed=9)
    out = check_against_oracle(w, ro, params, w["T"], BF16, ids, obs_env_ids=ids)
    print(name, out)
    ro.close()


@pytest.mark.parametrize("precision", [FP32, BF16])
def test_hand_worked_warehouse_steps_on_the_gpu(precision):
    """States written with set_state, actions forced: pick-up, carrying, delivery with its replacement request, a
    carrying robot stopped by a shelf on the ground, a refused put-down in the delivery row, a head-on conflict."""
    import torch

    w = wl.workload(WH0)
    cfg = binding.make_config(w, precision=precision, max_T=1, n_envs=6)
    ro = binding.Rollout(cfg)
    params = torch.from_numpy(wl.make_params(w)).cuda()
    # record: r0(r,c,carry) r1(r,c,carry) s0(r,c,status) s1(r,c,status) step episode deliveries
    states = np.array([
        [3, 4, 0, 6, 0, 0, 3, 4, 2, 7, 7, 1, 0, 0, 0],   # robot 0 under shelf 0 picks it up
        [3, 4, 1, 6, 0, 0, 3, 4, 2, 7, 7, 1, 0, 0, 0],   # carries it up: the shelf moves along
        [1, 4, 1, 6, 0, 0, 1, 4, 2, 7, 7, 1, 5, 0, 0],   # into the delivery row: paid 1, shelf 1 takes the request
        [3, 3, 2, 6, 0, 0, 3, 4, 1, 3, 3, 2, 0, 0, 0],   # carrying robot stopped by the shelf on the ground to its right
        [0, 4, 1, 6, 0, 0, 0, 4, 1, 7, 7, 2, 0, 0, 0],   # no put-down in the delivery row
        [3, 2, 0, 3, 4, 0, 7, 7, 1, 6, 6, 2, 0, 0, 0],   # head-on: both stay
    ], dtype=np.int32)
    acts = np.array([[5, 0], [1, 0], [1, 0], [4, 0], [5, 0], [4, 3]], dtype=np.int32)[None]
    ro.set_state(states)
    ro.run_forced(params, 1, torch.from_numpy(acts).cuda())
    assert ro.status() == 0
    after = ro.get_state()
    assert after[0, :3].tolist() == [3, 4, 1] and after[0, 6:9].tolist() == [3, 4, 2]
    assert after[1, :3].tolist() == [2, 4, 1] and after[1, 6:9].tolist() == [2, 4, 2]
    assert after[2, :3].tolist() == [0, 4, 1] and after[2, 6:9].tolist() == [0, 4, 1] and after[2, 9:12].tolist() == [7, 7, 2]
    assert after[2, 14] == 1 and ro.rewards[0, 2].cpu().numpy().tolist() == [1.0, 1.0]
    assert after[3, :3].tolist() == [3, 3, 2] and after[3, 9:12].tolist() == [3, 3, 2]
    assert after[4, :3].tolist() == [0, 4, 1]
    assert after[5, :6].tolist() == [3, 2, 0, 3, 4, 0]
    assert ro.dones[0].cpu().numpy().tolist() == [0] * 6
    assert float(ro.rewards[0].sum()) == 2.0


@pytest.mark.parametrize("precision", [FP32, BF16])
@pytest.mark.parametrize("name,n_envs", [(WH0, 16), (WH2, 130)])
def test_warehouse_evaluation_block(name, n_envs, precision):
    """A greedy evaluation block of the warehouse family: episode counts, return sums, length sums and final states bit
    for bit against the oracle's transition under the GPU's own actions."""
    import torch

    from test_gpu_evaluate import _episode_sums, _state_records

    w = wl.workload(name)
    T = 130
    params = torch.from_numpy(wl.make_params(w, bias_scale=0.1)).cuda()
    ro = binding.Rollout(binding.make_config(w, precision=precision, max_T=4, n_envs=n_envs))
    cnt, ret, ln, acts = ro.evaluate(params, T, greedy=True, want_actions=True)
    assert ro.status() == binding.MAVA_OK
    acts = acts.cpu().numpy()
    env = oracle.rollout(oracle.make_config(w), w["seed"], None, T, np.arange(n_envs), forced_actions=acts, compute_mlp=False,
                         want_obs=False)
    c0, r0, l0 = _episode_sums(env.rewards, env.dones)
    assert np.array_equal(cnt.cpu().numpy(), c0) and np.array_equal(ln.cpu().numpy(), l0)
    assert np.array_equal(ret.cpu().numpy().view(np.uint32), r0.view(np.uint32))
    assert np.array_equal(ro.get_state(), _state_records(env.states, w["n_agents"], w["n_food"]))
    assert c0.sum() >= n_envs  # at least the cap ends an episode per environment
    ro.close()


def test_warehouse_shards_reproduce_the_whole_batch():
    """Two handles with first_env offsets give the bytes of one handle over all environments (Philox, the replacement
    requests included, is keyed on global environment indices)."""
    import torch

    w = wl.workload(WH2)
    T, n, cut = 40, 90, 37
    params = torch.from_numpy(wl.make_params(w)).cuda()
    whole = binding.Rollout(binding.make_config(w, precision=BF16, max_T=T, n_envs=n))
    lo = binding.Rollout(binding.make_config(w, precision=BF16, max_T=T, n_envs=cut))
    hi = binding.Rollout(binding.make_config(w, precision=BF16, max_T=T, n_envs=n - cut, first_env=cut))
    for r in (whole, lo, hi):
        r.run(params, T)
    for name in ("obs", "actions", "rewards", "dones", "logp", "values"):
        full = getattr(whole, name)
        assert torch.equal(full[:, :cut], getattr(lo, name)) and torch.equal(full[:, cut:], getattr(hi, name)), name
