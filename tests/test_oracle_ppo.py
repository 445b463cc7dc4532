"""Pins of the update-block oracle (oracle/ppo.py): the multi-agent PPO loss, its gradient, Adam.

Referees that are not the oracle's own formulas: float64 autograd of the loss written with torch
primitives, central finite differences of the loss value, closed forms, torch.optim.Adam and
torch.nn.utils.clip_grad_norm_.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import ppo
from paper_2107_01460_b200 import workloads as wl


def _random_batch(rng, R, D, N, net_kind, spread=1.0):
    """Rows whose ratios fall on both sides of the clip range and whose values fall inside and outside it."""
    b = {"obs": rng.standard_normal((R, D)), "actions": rng.integers(0, 6, R),
         "logp_old": np.log(1 / 6) + spread * 0.4 * rng.standard_normal(R), "adv": rng.standard_normal(R) * 2 + 0.3}
    S = R if net_kind == 0 else R // N
    if net_kind == 1:
        b["joint_obs"] = b["obs"].reshape(S, N * D)
    b["value_old"] = rng.standard_normal(S) * 0.5
    b["ret"] = rng.standard_normal(S)
    return b


def _setup(net_kind, seed=0, R=48, D=9, H=16, N=4):
    rng = np.random.default_rng(seed)
    shapes = ppo.layer_shapes(D, H, N, net_kind)
    n = sum(o * i + o for _, (o, i) in shapes)
    params = rng.standard_normal(n) * 0.25
    return rng, shapes, params, _random_batch(rng, R, D, N, net_kind)


def _torch_loss(params_t, shapes, net_kind, batch, hp):
    """The same loss, written independently with torch primitives (F.linear, log_softmax, clamp, minimum)."""
    F = torch.nn.functional
    off, layers = 0, []
    for _, (o, i) in shapes:
        W = params_t[off:off + o * i].reshape(o, i); off += o * i
        b = params_t[off:off + o]; off += o
        layers.append((W, b))
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    h = F.relu(F.linear(F.relu(F.linear(t(batch["obs"]), *layers[0])), *layers[1]))
    logits = F.linear(h, *layers[2])
    if net_kind == 0:
        values = F.linear(h, *layers[3])[:, 0]
    else:
        g = F.relu(F.linear(F.relu(F.linear(t(batch["joint_obs"]), *layers[3])), *layers[4]))
        values = F.linear(g, *layers[5])[:, 0]
    dist = torch.distributions.Categorical(logits=logits)
    logp = dist.log_prob(torch.from_numpy(np.asarray(batch["actions"])))
    ratio = torch.exp(logp - t(batch["logp_old"]))
    adv = t(batch["adv"])
    adv = (adv - adv.mean()) / (adv.std(unbiased=False) + 1e-8)
    actor = -torch.minimum(ratio * adv, torch.clamp(ratio, 1 - hp.clip_eps, 1 + hp.clip_eps) * adv).mean()
    v_old, ret = t(batch["value_old"]), t(batch["ret"])
    v_clip = v_old + torch.clamp(values - v_old, -hp.clip_eps, hp.clip_eps)
    value = 0.5 * torch.maximum((values - ret) ** 2, (v_clip - ret) ** 2).mean()
    return actor - hp.ent_coef * dist.entropy().mean() + hp.vf_coef * value, actor, dist.entropy().mean(), value


@pytest.mark.parametrize("net_kind", [0, 1])
def test_loss_and_gradient_against_float64_autograd(net_kind):
    hp = ppo.Hyper()
    rng, shapes, params, batch = _setup(net_kind)
    p_t = torch.from_numpy(params.copy()).requires_grad_(True)
    total, actor, ent, value = _torch_loss(p_t, shapes, net_kind, batch, hp)
    total.backward()
    got = ppo.ppo_loss(params, shapes, net_kind, batch, hp)
    assert abs(got["total"] - total.item()) < 1e-12 and abs(got["actor"] - actor.item()) < 1e-12
    assert abs(got["entropy"] - ent.item()) < 1e-12 and abs(got["value"] - value.item()) < 1e-12
    assert 0.1 < got["clip_frac"] < 0.95  # the batch exercises both branches of the clip
    grad = ppo.ppo_grad(params, shapes, net_kind, batch, hp)
    ref = p_t.grad.numpy()
    assert np.max(np.abs(grad - ref)) < 1e-12 * max(1.0, np.max(np.abs(ref)))
    assert np.count_nonzero(ref) > 0.5 * ref.size


@pytest.mark.parametrize("net_kind", [0, 1])
def test_gradient_against_central_differences_of_the_loss(net_kind):
    hp = ppo.Hyper(ent_coef=0.05, vf_coef=0.7)
    rng, shapes, params, batch = _setup(net_kind, seed=3)
    grad = ppo.ppo_grad(params, shapes, net_kind, batch, hp)
    for k in rng.choice(params.size, 40, replace=False):
        e = np.zeros_like(params); e[k] = 1e-6
        fd = (ppo.ppo_loss(params + e, shapes, net_kind, batch, hp)["total"] -
              ppo.ppo_loss(params - e, shapes, net_kind, batch, hp)["total"]) / 2e-6
        assert abs(fd - grad[k]) < 1e-6 * max(1.0, abs(grad[k])), (k, fd, grad[k])


def test_closed_forms_at_ratio_one_and_for_clipped_rows():
    rng, shapes, params, batch = _setup(0, seed=5)
    # rho = 1 everywhere: the surrogate is -mean(Ahat) = 0 whatever the policy, and a uniform policy has entropy log 6
    logits, values = ppo.forward(params, shapes, 0, batch["obs"])
    lp = logits - logits.max(1, keepdims=True)
    lp = lp - np.log(np.exp(lp).sum(1, keepdims=True))
    batch["logp_old"] = lp[np.arange(lp.shape[0]), batch["actions"]]
    got = ppo.ppo_loss(params, shapes, 0, batch)
    assert abs(got["actor"]) < 1e-12 and got["clip_frac"] == 0.0
    zero = np.zeros_like(params)
    assert abs(ppo.ppo_loss(zero, shapes, 0, batch)["entropy"] - np.log(6.0)) < 1e-12
    # value term alone, returns equal to old values and predictions inside the clip range: 0.5 * mean((V - R)^2)
    hp = ppo.Hyper(ent_coef=0.0, vf_coef=1.0)
    batch["value_old"] = values + 0.05
    batch["ret"] = values + 0.05
    assert abs(ppo.ppo_loss(params, shapes, 0, batch, hp)["value"] - 0.5 * 0.05 ** 2) < 1e-12
    # rows pushed outside the clip range on the side the clip cuts contribute nothing to the actor gradient: with every
    # ratio at 3, rows of positive advantage are clipped and only those of negative advantage keep their gradient
    batch["logp_old"] = batch["logp_old"] - np.log(3.0)            # rho = 3 > 1 + eps on every row
    hp = ppo.Hyper(ent_coef=0.0, vf_coef=0.0)
    g_all = ppo.ppo_grad(params, shapes, 0, batch, hp)
    keep = ppo.normalise(batch["adv"]) < 0                          # only rows with negative advantage stay unclipped
    # the same gradient from the unclipped rows alone, by autograd of -sum(rho Ahat)/R over those rows
    p_t = torch.from_numpy(params.copy()).requires_grad_(True)
    F = torch.nn.functional
    off, layers = 0, []
    for _, (o, i) in shapes:
        W = p_t[off:off + o * i].reshape(o, i); off += o * i
        b = p_t[off:off + o]; off += o
        layers.append((W, b))
    h = F.relu(F.linear(F.relu(F.linear(torch.from_numpy(batch["obs"]), *layers[0])), *layers[1]))
    logp = torch.log_softmax(F.linear(h, *layers[2]), -1)[torch.arange(keep.size), torch.from_numpy(batch["actions"])]
    rho = torch.exp(logp - torch.from_numpy(batch["logp_old"]))
    ahat = torch.from_numpy(ppo.normalise(batch["adv"]))
    (-(rho * ahat)[torch.from_numpy(keep)].sum() / keep.size).backward()
    assert np.max(np.abs(g_all - p_t.grad.numpy())) < 1e-10 * max(1.0, np.max(np.abs(g_all)))


def test_adam_and_global_norm_clipping_against_torch():
    hp = ppo.Hyper(lr=1e-2, max_grad_norm=0.5)
    rng = np.random.default_rng(7)
    p0 = rng.standard_normal(37)
    grads = [rng.standard_normal(37) * s for s in (3.0, 0.01, 1.0)]      # clipped, untouched, clipped
    p_t = torch.nn.Parameter(torch.from_numpy(p0.copy()))
    opt = torch.optim.Adam([p_t], lr=hp.lr, betas=(hp.beta1, hp.beta2), eps=hp.adam_eps)
    p, m, v = p0.copy(), np.zeros(37), np.zeros(37)
    for step, g in enumerate(grads, start=1):
        p_t.grad = torch.from_numpy(g.copy())
        torch.nn.utils.clip_grad_norm_([p_t], hp.max_grad_norm)
        opt.step()
        p, m, v = ppo.adam_step(p, g, m, v, step, hp)
        assert np.max(np.abs(p - p_t.detach().numpy())) < 1e-9
    g, norm = ppo.clip_by_global_norm(grads[1], hp.max_grad_norm)
    assert norm < hp.max_grad_norm and np.array_equal(g, grads[1])
    g, norm = ppo.clip_by_global_norm(grads[0], hp.max_grad_norm)
    assert abs(np.linalg.norm(g) - hp.max_grad_norm) < 1e-12


@pytest.mark.parametrize("idx", [0, 3])
def test_a_rolled_out_trajectory_feeds_the_update_and_a_small_step_lowers_the_loss(idx):
    w = wl.workload(idx)
    cfg = oracle.make_config(w)
    E, T = 6, 12
    params = wl.make_params(w, bias_scale=0.1).astype(np.float64)
    ro = oracle.rollout(cfg, w["seed"], params.astype(np.float32), T, np.arange(E))
    adv, ret = oracle.gae(ro.values, ro.rewards, ro.dones, wl.GAMMA, wl.LAMBDA)
    shapes = ppo.layer_shapes(wl.obs_dim(w), w["hidden"], w["n_agents"], w["net_kind"])
    assert [s for _, s in shapes] == [s for _, s in wl.param_shapes(w)]
    batch = ppo.batch_from_rollout(ro.obs, ro.own_actions, ro.logp, ro.values, adv, ret, w["net_kind"])
    loss0 = ppo.ppo_loss(params, shapes, w["net_kind"], batch)
    # the stored log-probs are those of the rollout's own parameters: every ratio is 1 (to the oracle's fp32 outputs)
    assert loss0["clip_frac"] == 0.0 and abs(loss0["actor"]) < 1e-5
    grad = ppo.ppo_grad(params, shapes, w["net_kind"], batch)
    assert np.isfinite(grad).all() and np.linalg.norm(grad) > 0
    loss1 = ppo.ppo_loss(params - 1e-3 * grad / np.linalg.norm(grad), shapes, w["net_kind"], batch)
    assert loss1["total"] < loss0["total"]


# ---- bf16-operand mode -------------------------------------------------------------------------------------------

def test_bf16_round_is_the_cast_torch_makes():
    rng = np.random.default_rng(11)
    x = np.concatenate([rng.standard_normal(4000) * 10.0 ** rng.integers(-30, 30, 4000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.0e-39, 65280.0, -2.5e-8],  # two exact ties among them
                        np.float32(1.0) + np.arange(0, 64) * 2.0 ** -9])
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    got = ppo.bf16_round(x)
    assert np.array_equal(got, want)
    assert np.array_equal(ppo.bf16_round(got), got)  # idempotent


class _RoundForward(torch.autograd.Function):
    """y = bf16(x); the gradient passes through unchanged."""
    @staticmethod
    def forward(ctx, x):
        return x.to(torch.float32).to(torch.bfloat16).to(torch.float64)

    @staticmethod
    def backward(ctx, g):
        return g


class _RoundBackward(torch.autograd.Function):
    """y = x; the gradient that flows back through here is rounded to bf16."""
    @staticmethod
    def forward(ctx, x):
        return x.clone()

    @staticmethod
    def backward(ctx, g):
        return g.to(torch.float32).to(torch.bfloat16).to(torch.float64)


@pytest.mark.parametrize("net_kind", [0, 1])
def test_bf16_operand_mode_against_autograd_with_torch_bfloat16_casts(net_kind):
    """The rounding points of the bf16-operand mode, restated as a torch graph: operands cast to torch.bfloat16 on the
    way in (gradient passes), pre-activations and head outputs (before their bias) wrapped so that the gradient
    flowing back through them is cast to torch.bfloat16.  Autograd then yields what the oracle must compute."""
    hp = ppo.Hyper()
    rng, shapes, params, batch = _setup(net_kind, seed=21, R=64)
    # gradients of a realistic size (the 1/R of the mean and small derivatives): bf16 keeps the exponent
    F = torch.nn.functional
    rf, rb = _RoundForward.apply, _RoundBackward.apply
    p_t = torch.from_numpy(params.copy()).requires_grad_(True)
    off, layers = 0, []
    for _, (o, i) in shapes:
        W = p_t[off:off + o * i].reshape(o, i); off += o * i
        b = p_t[off:off + o]; off += o
        layers.append((W, b))
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))

    def torso(x, l1, l2):
        h1 = rf(F.relu(rb(F.linear(rf(x), rf(l1[0]), l1[1]))))
        return rf(F.relu(rb(F.linear(h1, rf(l2[0]), l2[1]))))

    h = torso(t(batch["obs"]), layers[0], layers[1])
    logits = rb(F.linear(h, rf(layers[2][0]))) + layers[2][1]
    if net_kind == 0:
        values = (rb(F.linear(h, rf(layers[3][0]))) + layers[3][1])[:, 0]
    else:
        g = torso(t(batch["joint_obs"]), layers[3], layers[4])
        values = (rb(F.linear(g, rf(layers[5][0]))) + layers[5][1])[:, 0]
    dist = torch.distributions.Categorical(logits=logits)
    logp = dist.log_prob(torch.from_numpy(np.asarray(batch["actions"])))
    ratio = torch.exp(logp - t(batch["logp_old"]))
    adv = t(batch["adv"])
    adv = (adv - adv.mean()) / (adv.std(unbiased=False) + 1e-8)
    actor = -torch.minimum(ratio * adv, torch.clamp(ratio, 1 - hp.clip_eps, 1 + hp.clip_eps) * adv).mean()
    v_old, ret = t(batch["value_old"]), t(batch["ret"])
    v_clip = v_old + torch.clamp(values - v_old, -hp.clip_eps, hp.clip_eps)
    value = 0.5 * torch.maximum((values - ret) ** 2, (v_clip - ret) ** 2).mean()
    total = actor - hp.ent_coef * dist.entropy().mean() + hp.vf_coef * value
    total.backward()
    got = ppo.ppo_loss(params, shapes, net_kind, batch, hp, emulate_bf16=True)
    assert abs(got["total"] - total.item()) < 1e-12 and abs(got["value"] - value.item()) < 1e-12
    grad = ppo.ppo_grad(params, shapes, net_kind, batch, hp, emulate_bf16=True)
    ref = p_t.grad.numpy()
    assert np.max(np.abs(grad - ref)) < 1e-12 * max(1.0, np.max(np.abs(ref)))
    # and the mode is a perturbation of the exact gradient of the size bf16 rounding gives, not something else
    exact = ppo.ppo_grad(params, shapes, net_kind, batch, hp)
    err = np.max(np.abs(grad - exact)) / np.max(np.abs(exact))
    assert 1e-5 < err < 0.15, err  # 64 rows: a single ratio that changes sides of a clip is visible


def test_bf16_operand_mode_changes_nothing_when_every_quantity_is_representable():
    """Weights, observations and hidden activations that are small integers are bf16 numbers already; with the loss
    reduced to the value term and targets that make every derivative a power of two, no rounding point changes a value
    and the mode must return the exact gradient."""
    D, H, R = 5, 4, 8
    shapes = ppo.layer_shapes(D, H, 2, 0)
    rng = np.random.default_rng(2)
    parts = []
    for _, (o, i) in shapes:
        parts += [rng.integers(-2, 3, (o, i)).astype(np.float64).ravel(), rng.integers(-1, 2, o).astype(np.float64)]
    params = np.concatenate(parts)
    batch = {"obs": rng.integers(0, 3, (R, D)).astype(np.float64), "actions": rng.integers(0, 6, R),
             "logp_old": np.full(R, np.log(1 / 6)), "adv": rng.standard_normal(R)}
    _, values = ppo.forward(params, shapes, 0, batch["obs"])
    batch["value_old"] = values.copy()
    batch["ret"] = values - 0.5                       # V - R = 1/2 on every row, inside the clip range
    hp = ppo.Hyper(ent_coef=0.0, vf_coef=1.0, clip_eps=0.2)
    only_value = dict(batch, adv=np.zeros(R) + 0.0)
    only_value["adv"] = np.array([1.0, -1.0] * (R // 2)) * 0.0  # zero advantages: the surrogate has no gradient
    a = ppo.ppo_grad(params, shapes, 0, only_value, hp)
    b = ppo.ppo_grad(params, shapes, 0, only_value, hp, emulate_bf16=True)
    assert np.abs(a).max() > 0 and np.array_equal(a, b)
