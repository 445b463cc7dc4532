"""Recurrent-policy rollout on the GPU (through the C ABI) against the oracle's recurrent rollout."""
import numpy as np
import pytest

import oracle
from paper_2107_01460_b200 import binding, workloads as wl

from parity import check_recurrent_against_oracle

pytestmark = pytest.mark.gpu
FP32, BF16 = binding.MAVA_PRECISION_FP32, binding.MAVA_PRECISION_BF16
REC0, REC1, REC2 = "rec0_tiny_8x8_2p2f_gru64", "rec1_8x8_2p2f_gru64", "rec2_10x10_3p3f_gru64"


def _run(w, precision, T, n_envs=None, bias_scale=0.1):
    import torch

    cfg = binding.make_config(w, precision=precision, flags=binding.MAVA_FLAG_WRITE_LOGITS, max_T=T, n_envs=n_envs)
    ro = binding.Rollout(cfg)
    params = wl.make_params(w, bias_scale=bias_scale)
    ro.run(torch.from_numpy(params).cuda(), T)
    ro.gae(np.float32(wl.GAMMA), np.float32(wl.LAMBDA))
    assert ro.status() == binding.MAVA_OK
    return ro, params


def _bf16_compiled(w):
    try:
        binding.Rollout(binding.make_config(w, precision=BF16, n_envs=2, max_T=1)).close()
        return True
    except binding.MavaError:
        return False


@pytest.mark.parametrize("precision", [FP32, BF16])
@pytest.mark.parametrize("name,n_envs,T", [(REC0, 16, 70), (REC2, 45, 120), (REC1, 1, 3), (REC2, 300, 40)])
def test_recurrent_rollout_every_environment(name, n_envs, T, precision):
    """T beyond the episode cap: every environment restarts inside the run, and with it its agents' memory."""
    w = wl.workload(name)
    if precision == BF16 and not _bf16_compiled(w):
        pytest.skip("recurrent policy: tensor-core kernel not compiled")
    ro, params = _run(w, precision, T, n_envs=n_envs)
    out = check_recurrent_against_oracle(w, ro, params, T, precision, np.arange(n_envs))
    print(name, precision, out)
    ro.close()


@pytest.mark.parametrize("precision", [FP32, BF16])
def test_two_calls_continue_like_one_and_reset_replays(precision):
    import torch

    w = wl.workload(REC1)
    if precision == BF16 and not _bf16_compiled(w):
        pytest.skip("recurrent policy: tensor-core kernel not compiled")
    cfg = binding.make_config(w, precision=precision, max_T=70, n_envs=40)
    params = torch.from_numpy(wl.make_params(w, bias_scale=0.1)).cuda()
    a = binding.Rollout(cfg)
    a.run(params, 70)
    b = binding.Rollout(cfg)
    b.run(params, 30)
    first = [t[:30].clone() for t in (b.obs, b.actions, b.logp, b.values)]
    b.run(params, 40)
    for x, y, z in zip(first, (b.obs, b.actions, b.logp, b.values), (a.obs, a.actions, a.logp, a.values)):
        assert torch.equal(z[:30], x) and torch.equal(z[30:70], y[:40])
    assert torch.equal(a.values[70], b.values[40])
    assert np.array_equal(a.get_hidden(), b.get_hidden()) and np.array_equal(a.get_state(), b.get_state())
    whole = [t.clone() for t in (a.obs, a.actions, a.logp, a.values)]
    a.reset(w["seed"])
    assert not a.get_hidden().any()
    a.run(params, 70)
    for x, y in zip(whole, (a.obs, a.actions, a.logp, a.values)):
        assert torch.equal(x, y)
    assert a.status() == 0 and b.status() == 0


@pytest.mark.parametrize("name", [REC1, REC2])
def test_recurrent_full_size(name):
    """The full-size recurrent workloads in the precision the benchmark times: environment arrays for every environment,
    the network on the first 64, the last 64 and 128 seeded-random environments at every step."""
    w = wl.workload(name)
    precision = BF16 if _bf16_compiled(w) else FP32
    ro, params = _run(w, precision, w["T"], bias_scale=0.0)
    ids = wl.sample_env_ids(w["n_envs"], 64, 64, 128, seed=5)
    out = check_recurrent_against_oracle(w, ro, params, w["T"], precision, ids)
    print(name, precision, out)
    ro.close()


def test_what_the_recurrent_policy_does_not_offer_is_refused():
    import torch

    w = wl.workload(REC0)
    ro = binding.Rollout(binding.make_config(w, precision=FP32))
    params = torch.from_numpy(wl.make_params(w)).cuda()
    ro.run(params, 4)
    ro.gae(wl.GAMMA, wl.LAMBDA)
    with pytest.raises(binding.MavaError) as e:
        ro.ppo_grad(params)
    assert e.value.code == binding.MAVA_ERR_UNSUPPORTED
    with pytest.raises(binding.MavaError) as e:
        ro.evaluate(params, 4)
    assert e.value.code == binding.MAVA_ERR_UNSUPPORTED
    ff = binding.Rollout(binding.make_config(wl.workload(0), precision=FP32))
    with pytest.raises(binding.MavaError):
        ff.get_hidden()
