"""The give-up path of the kernels' bounded waits, exercised without faulting, trapping or hanging anything: one armed
launch makes one thread block wait briefly on a barrier phase that nothing completes, at a point where none of its
copies or MMAs is outstanding.  The block must record the time-out and leave in order (copies drained, tensor memory
freed, its partner thread group walked through the hand-over protocol), the status call must report it once, and the
same handle must work again afterwards."""
import numpy as np
import pytest

from paper_2107_01460_b200 import binding, workloads as wl

from parity import check_against_oracle

pytestmark = pytest.mark.gpu
BF16 = binding.MAVA_PRECISION_BF16


def _fresh_run_matches(w, ro, params, p_dev, T, ids):
    ro.reset(w["seed"])
    ro.run(p_dev, T)
    ro.gae(np.float32(wl.GAMMA), np.float32(wl.LAMBDA))
    assert ro.status() == binding.MAVA_OK
    check_against_oracle(w, ro, params, T, BF16, ids)


def test_gae_copy_engine_kernel_gives_up_and_recovers():
    import torch

    w = wl.workload(2)
    T, n_envs = 32, 5488  # 16 464 columns: the persistent copy-engine kernel
    params = wl.make_params(w)
    ro = binding.Rollout(binding.make_config(w, precision=BF16, max_T=T, n_envs=n_envs, flags=binding.MAVA_FLAG_WRITE_LOGITS))
    p_dev = torch.from_numpy(params).cuda()
    ro.run(p_dev, T)
    ro.debug_expire_next_wait(binding.MAVA_EXPIRE_GAE)
    ro.gae(wl.GAMMA, wl.LAMBDA)
    assert ro.status() == binding.MAVA_ERR_DEVICE_TIMEOUT
    assert ro.status() == binding.MAVA_OK  # reported once
    _fresh_run_matches(w, ro, params, p_dev, T, wl.sample_env_ids(n_envs, 4, 4, 8, seed=7))


@pytest.mark.parametrize("idx,n_envs", [(4, 1200), (2, 5000)])
def test_rollout_kernel_gives_up_and_recovers(idx, n_envs):
    """idx 4: the two thread groups of an SM share one tile set and hand it to each other through named barriers; the
    group that gives up, and its partner once it sees the flag, must keep walking that protocol to the end.
    idx 2: independent groups; the one that gives up simply stops."""
    import torch

    w = wl.workload(idx)
    T = 24
    params = wl.make_params(w)
    ro = binding.Rollout(binding.make_config(w, precision=BF16, max_T=T, n_envs=n_envs, flags=binding.MAVA_FLAG_WRITE_LOGITS))
    p_dev = torch.from_numpy(params).cuda()
    ro.debug_expire_next_wait(binding.MAVA_EXPIRE_ROLLOUT)
    ro.run(p_dev, T)
    assert ro.status() == binding.MAVA_ERR_DEVICE_TIMEOUT
    assert ro.status() == binding.MAVA_OK
    _fresh_run_matches(w, ro, params, p_dev, T, wl.sample_env_ids(n_envs, 4, 4, 8, seed=7))


def test_gae_longer_than_its_limit_is_a_capacity_error():
    import torch

    w = wl.workload(0)
    T = binding.MAVA_GAE_MAX_T + 1
    ro = binding.Rollout(binding.make_config(w, precision=binding.MAVA_PRECISION_FP32, max_T=T, n_envs=4))
    ro.run(torch.from_numpy(wl.make_params(w)).cuda(), T)
    with pytest.raises(binding.MavaError) as e:
        ro.gae(wl.GAMMA, wl.LAMBDA)
    assert e.value.code == binding.MAVA_ERR_CAPACITY
    assert ro.status() == binding.MAVA_OK
