"""GPU evaluation block (mava_rollout_evaluate) against the oracle.

A single different action changes the rest of an episode, so the block is checked the way the
rollout is: the environment side and the episode sums bit for bit under the GPU's own actions, and
every greedy action as a valid arg max of the oracle's logits for the same state (equal unless
the two best logits lie within the path's tolerance of each other)."""
import numpy as np
import pytest

import oracle
from parity import TOL
from paper_2107_01460_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu
FP32, BF16 = binding.MAVA_PRECISION_FP32, binding.MAVA_PRECISION_BF16


def _state_records(states, N, F):
    return np.array([[*sum(([s.agent_r[n], s.agent_c[n], s.agent_level[n]] for n in range(N)), []),
                      *sum(([s.food_r[f], s.food_c[f], s.food_level[f]] for f in range(F)), []),
                      s.step, s.episode, s.total_food_level] for s in states], dtype=np.int32)


def _episode_sums(rewards, dones):
    T, n = dones.shape
    cnt, ret, ln = np.zeros(n, np.int32), np.zeros(n, np.float32), np.zeros(n, np.int32)
    for e in range(n):
        run, length = np.float32(0), 0
        for t in range(T):
            run = np.float32(run + rewards[t, e, 0])
            length += 1
            if dones[t, e]:
                cnt[e] += 1
                ret[e] = np.float32(ret[e] + run)
                ln[e] += length
                run, length = np.float32(0), 0
    return cnt, ret, ln


def _check_block(w, precision, n_envs, T, mlp_ids, flags=0):
    import torch

    params = wl.make_params(w, bias_scale=0.1)
    p_dev = torch.from_numpy(params).cuda()
    ro = binding.Rollout(binding.make_config(w, precision=precision, max_T=4, n_envs=n_envs, flags=flags))
    cnt, ret, ln, acts = ro.evaluate(p_dev, T, greedy=True, want_actions=True)
    assert ro.status() == binding.MAVA_OK
    cnt, ret, ln, acts = cnt.cpu().numpy(), ret.cpu().numpy(), ln.cpu().numpy(), acts.cpu().numpy()
    assert acts.min() >= 0 and acts.max() < 6
    ocfg = oracle.make_config(w)
    # environment side under the GPU's actions, every environment: sums and final states bit for bit
    env = oracle.rollout(ocfg, w["seed"], None, T, np.arange(n_envs), forced_actions=acts, compute_mlp=False,
                         want_obs=False)
    c0, r0, l0 = _episode_sums(env.rewards, env.dones)
    assert np.array_equal(cnt, c0) and np.array_equal(ln, l0)
    assert np.array_equal(ret.view(np.uint32), r0.view(np.uint32))
    assert np.array_equal(ro.get_state(), _state_records(env.states, w["n_agents"], w["n_food"]))
    # the oracle's own block on a few environments: same sums, and the GPU's actions are arg maxes
    ids = np.asarray(mlp_ids, dtype=np.int32)
    ev = oracle.evaluate(ocfg, w["seed"], params, T, ids, forced_actions=acts[:, ids],
                         emulate_bf16=(precision == BF16))
    assert np.array_equal(ev.ep_count, cnt[ids]) and np.array_equal(ev.len_sum, ln[ids])
    assert np.array_equal(ev.ret_sum.view(np.uint32), ret[ids].view(np.uint32))
    top = ev.logits.max(axis=-1)
    chosen = np.take_along_axis(ev.logits, acts[:, ids][..., None], axis=-1)[..., 0]
    tol = (2e-3 if precision == BF16 else TOL[FP32]) * 4.0 * (1.0 + np.abs(top))
    assert np.all(top - chosen <= tol), "a greedy action is not an arg max of the oracle's logits"
    same = float(np.mean(acts[:, ids] == np.argmax(ev.logits, axis=-1)))
    assert same > 0.97, same
    return int(cnt.sum())


@pytest.mark.parametrize("idx,precision,n_envs,T", [
    (0, FP32, 16, 120), (0, BF16, 16, 120), (1, FP32, 40, 110), (1, BF16, 333, 110), (1, BF16, 1500, 60),
    (2, BF16, 300, 210), (2, BF16, 3000, 120), (3, BF16, 200, 130), (4, BF16, 150, 110), (3, FP32, 30, 105)])
def test_greedy_block(idx, precision, n_envs, T):
    w = wl.workload(idx)
    ended = _check_block(w, precision, n_envs, T, wl.sample_env_ids(n_envs, 3, 3, 3, seed=idx))
    assert ended >= n_envs  # every environment finished at least one episode (T exceeds the cap)


def test_wide_tiles_and_tensor_memory_layouts():
    w = wl.workload(1)
    _check_block(w, BF16, 333, 70, [0, 100, 332], flags=binding.MAVA_FLAG_WIDE_TILES)
    _check_block(w, BF16, 333, 70, [0, 100, 332], flags=binding.MAVA_FLAG_HIDDEN_IN_TMEM)


@pytest.mark.parametrize("idx", [1, 4])
def test_full_size_block_in_the_benchmarks_launch_shape(idx):
    w = wl.workload(idx)
    E = w["n_envs"]
    _check_block(w, BF16, E, w["T"], wl.sample_env_ids(E, 2, 2, 2, seed=idx))


@pytest.mark.parametrize("idx,precision", [(0, FP32), (1, BF16), (4, BF16)])
def test_sampled_block_draws_the_rollouts_actions_and_blocks_chain(idx, precision):
    """greedy = 0 takes the rollout's draws; a block advances the handle like a run of the same length."""
    import torch

    w = wl.workload(idx)
    n, T1, T2 = 96, 70, 50
    params = torch.from_numpy(wl.make_params(w, bias_scale=0.1)).cuda()
    a = binding.Rollout(binding.make_config(w, precision=precision, max_T=T1 + T2, n_envs=n))
    b = binding.Rollout(binding.make_config(w, precision=precision, max_T=T1 + T2, n_envs=n))
    a.run(params, T1 + T2)
    obs_before = b.obs.clone()
    cnt, ret, ln, acts = b.evaluate(params, T1, greedy=False, want_actions=True)
    assert torch.equal(acts, a.actions[:T1])
    assert torch.equal(b.obs, obs_before)  # the caller's trajectory buffers are not touched
    c0, r0, l0 = _episode_sums(a.rewards[:T1].cpu().numpy(), a.dones[:T1].cpu().numpy())
    assert np.array_equal(cnt.cpu().numpy(), c0) and np.array_equal(ln.cpu().numpy(), l0)
    assert np.array_equal(ret.cpu().numpy().view(np.uint32), r0.view(np.uint32))
    b.run(params, T2)  # continues where the block stopped, step counter included
    assert torch.equal(b.actions[:T2], a.actions[T1:T1 + T2]) and torch.equal(b.obs[:T2], a.obs[T1:T1 + T2])
    assert np.array_equal(a.get_state(), b.get_state())
    assert a.status() == 0 and b.status() == 0


def test_argument_errors():
    import torch

    w = wl.workload(0)
    ro = binding.Rollout(binding.make_config(w, precision=FP32, max_T=4, n_envs=4))
    params = torch.from_numpy(wl.make_params(w)).cuda()
    out = torch.zeros(4, dtype=torch.int32, device="cuda")
    outf = torch.zeros(4, dtype=torch.float32, device="cuda")
    L = binding.lib()
    bad = binding.MAVA_ERR_INVALID_ARG
    assert L.mava_rollout_evaluate(ro.handle, params.data_ptr(), 0, 1, out.data_ptr(), outf.data_ptr(), out.data_ptr(), None) == bad
    assert L.mava_rollout_evaluate(ro.handle, params.data_ptr(), 5, 1, None, outf.data_ptr(), out.data_ptr(), None) == bad
    assert L.mava_rollout_evaluate(ro.handle, None, 5, 1, out.data_ptr(), outf.data_ptr(), out.data_ptr(), None) == bad
    # longer than max_T is fine: nothing of the trajectory is stored
    assert L.mava_rollout_evaluate(ro.handle, params.data_ptr(), 9, 1, out.data_ptr(), outf.data_ptr(), out.data_ptr(), None) == 0
    assert ro.status() == 0
