"""Update block on the GPU (mava_ppo_grad, mava_adam_step) against the float64 oracle (oracle/ppo.py).

The GPU rolls out and runs GAE; the oracle gets the GPU's own trajectory arrays as its minibatch, so the
comparison is of the update block alone.  The kernels compute in fp32, sums that decide a mean in double.
Tolerance: a gradient entry is a sum over R rows of products of O(1) factors, rounded in fp32 along the way
(relative error about sqrt(R) * 2^-24 of the largest partial sums), so entries must agree to
2e-4 * max|grad| and the loss terms to 1e-5 * (1 + |ref|).
"""
import numpy as np
import pytest

import oracle
from oracle import ppo
from paper_2107_01460_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

FP32, BF16 = binding.MAVA_PRECISION_FP32, binding.MAVA_PRECISION_BF16


def _rolled_out(idx, n_envs, T, precision, bias_scale=0.1, flags=binding.MAVA_FLAG_UPDATE_FP32):
    """A handle after run + gae.  By default a bf16 handle keeps the fp32 update block (the path most cases here
    check); flags=0 lets it take the tensor-core kernels."""
    import torch

    w = wl.workload(idx)
    cfg = binding.make_config(w, precision=precision, max_T=T, n_envs=n_envs, flags=flags)
    ro = binding.Rollout(cfg)
    params = torch.from_numpy(wl.make_params(w, bias_scale=bias_scale)).cuda()
    ro.run(params, T)
    ro.gae(wl.GAMMA, wl.LAMBDA)
    return w, ro, params


def _oracle_batch(w, ro, T):
    g = lambda name, n: getattr(ro, name)[:n].cpu().numpy().astype(np.float64)
    return ppo.batch_from_rollout(g("obs", T), ro.actions[:T].cpu().numpy(), g("logp", T), g("values", T + 1), g("adv", T),
                                  g("ret", T), w["net_kind"])


@pytest.mark.parametrize("idx,n_envs,T,precision", [(0, 16, 32, FP32), (1, 77, 20, FP32), (2, 50, 33, BF16), (3, 45, 17, BF16),
                                                    (3, 9, 5, FP32), (4, 21, 11, FP32),
                                                    (1, 1024, 128, BF16)])  # the size and precision the benchmark times
def test_loss_and_gradient_match_the_oracle(idx, n_envs, T, precision):
    import torch

    w, ro, params = _rolled_out(idx, n_envs, T, precision)
    # parameters a little away from the rollout's own, so that ratios leave 1 and some rows are clipped
    g = torch.Generator(device="cuda").manual_seed(idx)
    new = params + 0.6 * torch.randn(params.shape, generator=g, device="cuda") * params.std()
    hp = binding.ppo_defaults()
    terms, grad = ro.ppo_grad(new, hp)
    assert ro.status() == binding.MAVA_OK
    shapes = ppo.layer_shapes(wl.obs_dim(w), w["hidden"], w["n_agents"], w["net_kind"])
    batch = _oracle_batch(w, ro, T)
    p64 = new.cpu().numpy().astype(np.float64)
    ref = ppo.ppo_loss(p64, shapes, w["net_kind"], batch)
    ref_grad = ppo.ppo_grad(p64, shapes, w["net_kind"], batch)
    t = terms.cpu().numpy()
    for k, name in enumerate(("total", "actor", "entropy", "value")):
        assert abs(t[k] - ref[name]) <= 1e-5 * (1 + abs(ref[name])), (name, t[k], ref[name])
    assert ref["clip_frac"] > 0.0  # the case exercises the clipped branch
    gg = grad.cpu().numpy().astype(np.float64)
    assert np.max(np.abs(gg - ref_grad)) <= 2e-4 * np.max(np.abs(ref_grad)), np.max(np.abs(gg - ref_grad)) / np.max(np.abs(ref_grad))
    # every layer's gradient is there (no segment left at zero)
    off = 0
    for _, (o, i) in shapes:
        assert np.abs(gg[off:off + o * i]).max() > 0 and np.abs(gg[off + o * i:off + o * i + o]).max() > 0
        off += o * i + o
    # a second call gives the same bytes (fixed summation order)
    terms2, grad2 = ro.ppo_grad(new, hp)
    assert torch.equal(grad, grad2) and torch.equal(terms, terms2)
    ro.close()


def test_at_the_rollouts_own_parameters_every_ratio_is_one():
    w, ro, params = _rolled_out(0, 16, 32, FP32)
    terms, grad = ro.ppo_grad(params)
    t = terms.cpu().numpy()
    assert abs(t[1]) < 1e-5          # -mean(Ahat) = 0
    assert 0 < t[2] <= np.log(6.0) + 1e-6
    ro.close()


@pytest.mark.parametrize("idx", [0, 3])
def test_adam_steps_match_the_oracle_and_lower_the_loss(idx):
    import torch

    w, ro, params = _rolled_out(idx, 24, 16, FP32)
    hp = binding.ppo_defaults()
    hp.lr = 1e-3
    ohp = ppo.Hyper(lr=1e-3)
    shapes = ppo.layer_shapes(wl.obs_dim(w), w["hidden"], w["n_agents"], w["net_kind"])
    batch = _oracle_batch(w, ro, 16)
    p = params.clone()
    m, v = torch.zeros_like(p), torch.zeros_like(p)
    p64 = params.cpu().numpy().astype(np.float64)
    m64, v64 = np.zeros_like(p64), np.zeros_like(p64)
    first = None
    for step in range(1, 4):
        terms, grad = ro.ppo_grad(p, hp)
        first = terms[0].item() if first is None else first
        ro.adam_step(p, grad, m, v, step, hp)
        p64, m64, v64 = ppo.adam_step(p64, ppo.ppo_grad(p64, shapes, w["net_kind"], batch, ohp), m64, v64, step, ohp)
        # Adam divides by sqrt(v): entries whose gradient is tiny amplify rounding, so compare in units of the step size
        assert np.max(np.abs(p.cpu().numpy() - p64)) <= 0.02 * ohp.lr * step, np.max(np.abs(p.cpu().numpy() - p64)) / ohp.lr
    last, _ = ro.ppo_grad(p, hp)
    assert ro.status() == binding.MAVA_OK
    assert last[0].item() < first
    ro.close()


def test_argument_errors():
    import torch

    w = wl.workload(0)
    ro = binding.Rollout(binding.make_config(w, precision=FP32))
    params = torch.from_numpy(wl.make_params(w)).cuda()
    with pytest.raises(binding.MavaError):  # no run yet
        ro.ppo_grad(params)
    ro.run(params, 4)
    ro.gae(wl.GAMMA, wl.LAMBDA)
    hp = binding.ppo_defaults()
    grad = torch.zeros_like(params)
    L = binding.lib()
    assert L.mava_ppo_grad(ro.handle, None, hp, grad.data_ptr(), None) == binding.MAVA_ERR_INVALID_ARG
    assert L.mava_adam_step(ro.handle, params.data_ptr(), grad.data_ptr(), grad.data_ptr(), grad.data_ptr(), 0, hp) == binding.MAVA_ERR_INVALID_ARG
    ro.close()


@pytest.mark.parametrize("idx,n_envs,T", [(1, 60, 20), (3, 30, 9), (2, 41, 16)])
def test_minibatches_of_environments(idx, n_envs, T):
    """A shuffled subset of the environments as the minibatch: the oracle gets the same environments' columns."""
    import torch

    w, ro, params = _rolled_out(idx, n_envs, T, FP32)
    g = torch.Generator(device="cuda").manual_seed(7 + idx)
    new = params + 0.6 * torch.randn(params.shape, generator=g, device="cuda") * params.std()
    perm = torch.randperm(n_envs, generator=g, device="cuda").to(torch.int32)
    shapes = ppo.layer_shapes(wl.obs_dim(w), w["hidden"], w["n_agents"], w["net_kind"])
    p64 = new.cpu().numpy().astype(np.float64)
    total = np.zeros_like(p64)
    pieces = [perm[: n_envs // 3].contiguous(), perm[n_envs // 3:].contiguous()]
    for ids in pieces:
        terms, grad = ro.ppo_grad(new, env_ids=ids)
        assert ro.status() == binding.MAVA_OK
        sel = ids.cpu().numpy().astype(np.int64)
        take = lambda name, n: getattr(ro, name)[:n].cpu().numpy().astype(np.float64)[:, sel]
        batch = ppo.batch_from_rollout(take("obs", T), ro.actions[:T].cpu().numpy()[:, sel], take("logp", T), take("values", T + 1),
                                       take("adv", T), take("ret", T), w["net_kind"])
        ref = ppo.ppo_loss(p64, shapes, w["net_kind"], batch)
        ref_grad = ppo.ppo_grad(p64, shapes, w["net_kind"], batch)
        t = terms.cpu().numpy()
        for k, name in enumerate(("total", "actor", "entropy", "value")):
            assert abs(t[k] - ref[name]) <= 1e-5 * (1 + abs(ref[name])), (name, t[k], ref[name])
        assert np.max(np.abs(grad.cpu().numpy() - ref_grad)) <= 2e-4 * np.max(np.abs(ref_grad))
    # all environments in order as the "minibatch" = the plain call, bit for bit
    ident = torch.arange(n_envs, dtype=torch.int32, device="cuda")
    t1, g1 = ro.ppo_grad(new)
    t2, g2 = ro.ppo_grad(new, env_ids=ident)
    assert torch.equal(g1, g2) and torch.equal(t1, t2)
    # an index out of range is reported, not followed
    bad = ident.clone()
    bad[3] = n_envs
    ro.ppo_grad(new, env_ids=bad)
    assert ro.status() == binding.MAVA_ERR_INVALID_ARG
    assert ro.status() == binding.MAVA_OK
    ro.close()


# ---- tensor-core path (bf16 handles, shared torso, H <= 128) ----------------------------------------------------------
# Tolerances.  Against the oracle in bf16-operand mode (same rounding points): every product of two bf16 numbers is
# exact in the fp32 accumulator, so what is left is the order of the fp32 additions (about sqrt(R) * 2^-24 of the
# largest partial sum), hidden activations that land on the other side of a bf16 rounding boundary (a fraction of
# about 2^-24 / 2^-8 of the elements, one bf16 ulp each) and rows whose ratio or value sits within fp32 rounding of a
# clip boundary (each worth 1/R of the gradient): 2e-3 * max|grad| and 2e-4 * (1 + |ref|) on the loss terms bound
# these with a wide margin.  Against the exact float64 oracle the operands' rounding itself shows (2^-9 relative per
# operand, logits good to 2e-2): 5e-2 * max|grad| and 2e-2 * (1 + |ref|).

def _tensor_path_reference(w, shapes, p64, batch, hp, emulate):
    """Oracle loss terms and gradient for the tensor-core path (with a centralised critic both nets take it)."""
    ref = ppo.ppo_loss(p64, shapes, w["net_kind"], batch, emulate_bf16=emulate)
    ref_grad = ppo.ppo_grad(p64, shapes, w["net_kind"], batch, emulate_bf16=emulate)
    return ref, ref_grad


@pytest.mark.parametrize("idx,n_envs,T", [(0, 16, 32), (1, 77, 20), (2, 50, 33), (2, 300, 40), (0, 1, 3),
                                          (1, 1024, 128),  # the size the benchmark times
                                          # H = 256: row kernel + weight kernel (with the centralised critic: both nets,
                                          # the critic's first layer one agent's observation at a time)
                                          (4, 21, 11), (4, 150, 40), (3, 45, 17), (3, 300, 20), (4, 1, 2), (3, 2, 3)])
def test_tensor_core_update_matches_the_bf16_operand_oracle(idx, n_envs, T):
    import torch

    w, ro, params = _rolled_out(idx, n_envs, T, BF16, flags=0)
    assert binding.update_on_tensor_cores(ro.cfg)
    g = torch.Generator(device="cuda").manual_seed(idx)
    new = params + 0.6 * torch.randn(params.shape, generator=g, device="cuda") * params.std()
    hp = binding.ppo_defaults()
    terms, grad = ro.ppo_grad(new, hp)
    assert ro.status() == binding.MAVA_OK
    shapes = ppo.layer_shapes(wl.obs_dim(w), w["hidden"], w["n_agents"], w["net_kind"])
    batch = _oracle_batch(w, ro, T)
    p64 = new.cpu().numpy().astype(np.float64)
    t = terms.cpu().numpy()
    gg = grad.cpu().numpy().astype(np.float64)
    for emulate, g_tol, l_tol in ((True, 2e-3, 2e-4), (False, 5e-2, 2e-2)):
        ref, ref_grad = _tensor_path_reference(w, shapes, p64, batch, hp, emulate)
        for k, name in enumerate(("total", "actor", "entropy", "value")):
            assert abs(t[k] - ref[name]) <= l_tol * (1 + abs(ref[name])), (emulate, name, t[k], ref[name])
        if not emulate and n_envs * T * w["n_agents"] < 1024:
            # a few dozen rows: one row whose ratio lands on the other side of a clip boundary once the operands are
            # rounded is several percent of the gradient, so the comparison with exact arithmetic says nothing here
            continue
        worst = np.max(np.abs(gg - ref_grad)) / np.max(np.abs(ref_grad))
        assert worst <= g_tol, (emulate, worst)
        # layer by layer as well: a layer with small gradients must not hide behind the largest one.  Against exact
        # arithmetic only the weight matrices are judged this way: a head's bias gradient is one number, the sum of
        # the rows' signed derivatives, which nearly cancels, so its own size is no scale for the operands' rounding.
        off = 0
        for name, (o, i) in shapes:
            for lo, hi in ((off, off + o * i), (off + o * i, off + o * i + o)):
                if not emulate and hi - lo < 8:
                    continue
                seg = np.max(np.abs(ref_grad[lo:hi]))
                assert np.max(np.abs(gg[lo:hi] - ref_grad[lo:hi])) <= 5 * g_tol * seg + 1e-12, (emulate, name, lo)
            off += o * i + o
    terms2, grad2 = ro.ppo_grad(new, hp)
    assert torch.equal(grad, grad2) and torch.equal(terms, terms2)  # fixed summation order
    ro.close()


@pytest.mark.parametrize("idx,n_envs,T", [(1, 333, 20), (2, 141, 16), (4, 90, 12), (3, 70, 9)])
def test_tensor_core_update_on_minibatches_of_environments(idx, n_envs, T):
    import torch

    w, ro, params = _rolled_out(idx, n_envs, T, BF16, flags=0)
    g = torch.Generator(device="cuda").manual_seed(17 + idx)
    new = params + 0.6 * torch.randn(params.shape, generator=g, device="cuda") * params.std()
    perm = torch.randperm(n_envs, generator=g, device="cuda").to(torch.int32)
    shapes = ppo.layer_shapes(wl.obs_dim(w), w["hidden"], w["n_agents"], w["net_kind"])
    p64 = new.cpu().numpy().astype(np.float64)
    for ids in (perm[: n_envs // 3].contiguous(), perm[n_envs // 3:].contiguous()):
        terms, grad = ro.ppo_grad(new, env_ids=ids)
        assert ro.status() == binding.MAVA_OK
        sel = ids.cpu().numpy().astype(np.int64)
        take = lambda name, n: getattr(ro, name)[:n].cpu().numpy().astype(np.float64)[:, sel]
        batch = ppo.batch_from_rollout(take("obs", T), ro.actions[:T].cpu().numpy()[:, sel], take("logp", T), take("values", T + 1),
                                       take("adv", T), take("ret", T), w["net_kind"])
        ref, ref_grad = _tensor_path_reference(w, shapes, p64, batch, binding.ppo_defaults(), True)
        t = terms.cpu().numpy()
        for k, name in enumerate(("total", "actor", "entropy", "value")):
            assert abs(t[k] - ref[name]) <= 2e-4 * (1 + abs(ref[name])), (name, t[k], ref[name])
        assert np.max(np.abs(grad.cpu().numpy() - ref_grad)) <= 2e-3 * np.max(np.abs(ref_grad))
    ident = torch.arange(n_envs, dtype=torch.int32, device="cuda")
    t1, g1 = ro.ppo_grad(new)
    t2, g2 = ro.ppo_grad(new, env_ids=ident)
    assert torch.equal(g1, g2) and torch.equal(t1, t2)  # rows through the copy engine or gathered by loads: the same bytes
    bad = ident.clone()
    bad[3] = n_envs
    ro.ppo_grad(new, env_ids=bad)
    assert ro.status() == binding.MAVA_ERR_INVALID_ARG
    ro.close()


def test_at_unchanged_parameters_the_ratios_of_a_bf16_handle_stay_near_one():
    """logp and values stored by the bf16 rollout come from bf16 tensor-core arithmetic.  Re-evaluated by the update
    block at the same parameters, the ratio must be 1 up to that arithmetic's noise: the tensor-core update (same
    operand rounding as the rollout) keeps the surrogate within 1e-3 of zero and the clipped fraction at nothing;
    the fp32 update on the same handle sees the rollout's bf16 rounding as policy change (reported, bounded)."""
    out = {}
    for name, flags in (("tensor", 0), ("fp32", binding.MAVA_FLAG_UPDATE_FP32)):
        w, ro, params = _rolled_out(1, 256, 64, BF16, flags=flags)
        terms, _ = ro.ppo_grad(params)
        out[name] = abs(terms[1].item())
        ro.close()
    print(out)
    assert out["tensor"] < 1e-3
    assert out["fp32"] < 3e-2


@pytest.mark.parametrize("idx,precision", [(1, BF16), (0, FP32), (3, BF16)])
def test_update_loop_in_one_call_equals_the_calls_it_stands_for(idx, precision):
    """mava_ppo_update (passes x minibatches of gradient + Adam inside the library) against the same sequence issued call
    by call: same kernels on the same inputs, so parameters, moments and loss terms must be the same bytes."""
    import torch

    n_envs, T, epochs, mbs = 96, 12, 2, 3
    w, ro, params = _rolled_out(idx, n_envs, T, precision, flags=0)
    g = torch.Generator(device="cuda").manual_seed(3)
    perm = torch.stack([torch.randperm(n_envs, generator=g, device="cuda") for _ in range(epochs)]).to(torch.int32).contiguous()
    hp = binding.ppo_defaults()
    p1, m1, v1 = params.clone(), torch.zeros_like(params), torch.zeros_like(params)
    terms1 = ro.ppo_update(p1, m1, v1, perm, mbs, 1, hp)
    p2, m2, v2 = params.clone(), torch.zeros_like(params), torch.zeros_like(params)
    terms2, step = [], 0
    for e in range(epochs):
        for k in range(mbs):
            ids = perm[e, n_envs * k // mbs: n_envs * (k + 1) // mbs].contiguous()
            t, grad = ro.ppo_grad(p2, hp, env_ids=ids)
            step += 1
            ro.adam_step(p2, grad, m2, v2, step, hp)
            terms2.append(t.clone())
    assert ro.status() == binding.MAVA_OK
    assert torch.equal(p1, p2) and torch.equal(m1, m2) and torch.equal(v1, v2)
    assert torch.equal(terms1, torch.stack(terms2))
    assert not torch.equal(p1, params)
    ro.close()
