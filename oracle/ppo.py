"""CPU oracle of the update block: multi-agent PPO loss, its gradient and the optimiser step.

TEST INFRASTRUCTURE ONLY, like the rest of this package: plain numpy in float64, no blocking, no
fusion, one statement per formula.  Nothing under the CUDA package imports it.

What it follows.  The report (Section 2, "Strong baseline algorithms and training architectures",
Figure 2) says that every update function takes the rolled-out experience and minimises multi-agent
PPO losses, for independent learners (a critic head on the shared torso) and for a centralised
critic; it prints no formula and no coefficient.  The reading taken here is the clipped-surrogate
objective of Schulman et al. (2017) as multi-agent PPO systems commonly use it, over ONE minibatch of
rows (a row = one agent at one environment-step):

    rho_i   = exp(logp_new(a_i) - logp_old_i)
    Ahat_i  = (A_i - mean A) / (std A + 1e-8)                    (population std over the minibatch)
    L_actor = -mean_i min(rho_i Ahat_i, clip(rho_i, 1-eps, 1+eps) Ahat_i)
    H_i     = -sum_k p_ik log p_ik,  Hbar = mean_i H_i
    Vc_j    = Vold_j + clip(V_j - Vold_j, -eps, +eps)
    L_value = 0.5 * mean_j max((V_j - R_j)^2, (Vc_j - R_j)^2)
    L       = L_actor - c_ent * Hbar + c_val * L_value

with eps = 0.2, c_ent = 0.01, c_val = 0.5.  With the shared torso the value rows j are the actor rows
i; with the centralised critic a value row is one environment-step (its input the agents'
observations concatenated, its target and old value those of agent 0's slot, all slots being equal).
The optimiser is Adam (Kingma & Ba 2015) with bias correction, after scaling the gradient so that
its global 2-norm is at most `max_grad_norm`.

bf16-operand mode (`emulate_bf16=True`).  The tensor-core kernels of the update block multiply bf16 operands and
accumulate in fp32; this mode states which quantities are rounded to bf16 (round to nearest even) and where, so
that those kernels can be compared tightly: the observations x, the weights W1, W2 and the head weights as
operands of every product (biases stay unrounded and are added to the accumulated sum); the hidden activations
h1 = bf16(relu(z1)) and h2 = bf16(relu(z2)); the per-row derivatives of the loss with respect to the six logits
and the value, rounded before they enter the products d h2 = dhead . Wh and d Wh = dhead^T . h2 (the head-bias
gradients sum the unrounded derivatives); d z2 = bf16(d h2 * [h2 > 0]) and d z1 = bf16(d h1 * [h1 > 0]) before
d W = d z^T . (input), d b = sum d z and d h1 = d z2 . W2.  Everything else (softmax, ratios, clips, means) is
not rounded.  This is a reading of how a bf16 tensor-core path rounds, not something the report states.

Pins (tests/test_oracle_ppo.py): float64 autograd of the same loss written with torch primitives as
referee, central finite differences of `ppo_loss` (no autograd involved), the closed forms at
rho = 1, the zero gradient of clipped rows, `torch.optim.Adam` and `clip_grad_norm_`.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

N_ACTIONS = 6


@dataclass
class Hyper:
    clip_eps: float = 0.2
    ent_coef: float = 0.01
    vf_coef: float = 0.5
    lr: float = 2.5e-4
    beta1: float = 0.9
    beta2: float = 0.999
    adam_eps: float = 1e-5
    max_grad_norm: float = 0.5


def layer_shapes(obs_dim: int, hidden: int, n_agents: int, net_kind: int):
    """(name, (out, in)) in the order of the flat parameter array (weight [out][in], then bias)."""
    layers = [("W1", (hidden, obs_dim)), ("W2", (hidden, hidden)), ("Wa", (N_ACTIONS, hidden))]
    if net_kind == 0:
        layers += [("Wv", (1, hidden))]
    else:
        layers += [("C1", (hidden, n_agents * obs_dim)), ("C2", (hidden, hidden)), ("Cv", (1, hidden))]
    return layers


def unpack(params: np.ndarray, shapes):
    """Views [(W, b), ...] into a flat float64 parameter (or gradient) array."""
    out, off = [], 0
    for _, (o, i) in shapes:
        W = params[off:off + o * i].reshape(o, i)
        off += o * i
        b = params[off:off + o]
        off += o
        out.append((W, b))
    assert off == params.size
    return out


def bf16_round(x):
    """float64 array -> the nearest bfloat16 values (ties to even), as float64.  Written on the bit pattern of
    binary32: add 0x7FFF plus the lowest kept bit, drop the low 16 bits."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def _r(x, emulate_bf16):
    return bf16_round(x) if emulate_bf16 else x


def _forward_torso(x, W1, b1, W2, b2, emulate_bf16=False):
    """z1, h1, z2, h2 of the two hidden layers; in bf16-operand mode x, W1, W2 arrive rounded and h1, h2 are rounded here."""
    z1 = x @ W1.T + b1
    h1 = _r(np.maximum(z1, 0.0), emulate_bf16)
    z2 = h1 @ W2.T + b2
    h2 = _r(np.maximum(z2, 0.0), emulate_bf16)
    return z1, h1, z2, h2


def forward(params, shapes, net_kind, obs, joint_obs=None, emulate_bf16=False):
    """logits [R][6] and values (shared torso: [R]; centralised critic: [S] over `joint_obs`)."""
    e = emulate_bf16
    p = unpack(np.asarray(params, dtype=np.float64), shapes)
    (W1, b1), (W2, b2), (Wa, ba) = p[0], p[1], p[2]
    _, _, _, h2 = _forward_torso(_r(obs, e), _r(W1, e), b1, _r(W2, e), b2, e)
    logits = h2 @ _r(Wa, e).T + ba
    if net_kind == 0:
        (Wv, bv) = p[3]
        values = (h2 @ _r(Wv, e).T + bv)[:, 0]
    else:
        (C1, c1), (C2, c2), (Cv, cv) = p[3], p[4], p[5]
        _, _, _, g2 = _forward_torso(_r(joint_obs, e), _r(C1, e), c1, _r(C2, e), c2, e)
        values = (g2 @ _r(Cv, e).T + cv)[:, 0]
    return logits, values


def _log_softmax(z):
    m = z.max(axis=1, keepdims=True)
    s = z - m
    return s - np.log(np.exp(s).sum(axis=1, keepdims=True))


def normalise(adv):
    adv = np.asarray(adv, dtype=np.float64)
    return (adv - adv.mean()) / (adv.std() + 1e-8)


def ppo_loss(params, shapes, net_kind, batch, hp: Hyper = Hyper(), emulate_bf16=False):
    """The loss terms of one minibatch.  `batch`: obs [R][D], actions [R], logp_old [R], adv [R] and,
    for the value rows, value_old, ret (shared torso: [R]; centralised: [S] with joint_obs [S][N*D])."""
    obs = np.asarray(batch["obs"], dtype=np.float64)
    logits, values = forward(params, shapes, net_kind, obs, batch.get("joint_obs"), emulate_bf16)
    a = np.asarray(batch["actions"], dtype=np.int64)
    logp_all = _log_softmax(logits)
    logp = logp_all[np.arange(a.size), a]
    rho = np.exp(logp - np.asarray(batch["logp_old"], dtype=np.float64))
    ahat = normalise(batch["adv"])
    surr = np.minimum(rho * ahat, np.clip(rho, 1.0 - hp.clip_eps, 1.0 + hp.clip_eps) * ahat)
    actor = -surr.mean()
    entropy = (-(np.exp(logp_all) * logp_all).sum(axis=1)).mean()
    v_old = np.asarray(batch["value_old"], dtype=np.float64)
    ret = np.asarray(batch["ret"], dtype=np.float64)
    v_clip = v_old + np.clip(values - v_old, -hp.clip_eps, hp.clip_eps)
    value = 0.5 * np.maximum((values - ret) ** 2, (v_clip - ret) ** 2).mean()
    total = actor - hp.ent_coef * entropy + hp.vf_coef * value
    return {"total": total, "actor": actor, "entropy": entropy, "value": value,
            "clip_frac": float(np.mean(np.abs(rho - 1.0) > hp.clip_eps))}


def _backward_torso(x, z1, h1, z2, h2, dh2, W2, emulate_bf16=False):
    """Gradients of the two hidden layers given dL/dh2; returns (dW1, db1, dW2, db2).  The ReLU gates are
    [z > 0]; in bf16-operand mode they are [h > 0] of the rounded activations (the same set unless a positive z
    rounds to zero, below 1e-40) and d z2, d z1 are rounded before every use."""
    dz2 = _r(dh2 * ((h2 if emulate_bf16 else z2) > 0.0), emulate_bf16)
    dW2 = dz2.T @ h1
    db2 = dz2.sum(axis=0)
    dh1 = dz2 @ W2
    dz1 = _r(dh1 * ((h1 if emulate_bf16 else z1) > 0.0), emulate_bf16)
    dW1 = dz1.T @ x
    db1 = dz1.sum(axis=0)
    return dW1, db1, dW2, db2


def ppo_grad(params, shapes, net_kind, batch, hp: Hyper = Hyper(), emulate_bf16=False):
    """dL/dparams as a flat float64 array in the parameter order, by the chain rule written out."""
    e = emulate_bf16
    params = np.asarray(params, dtype=np.float64)
    p = unpack(params, shapes)
    (W1, b1), (W2, b2), (Wa, ba) = p[0], p[1], p[2]
    W1, W2, Wa = _r(W1, e), _r(W2, e), _r(Wa, e)
    x = _r(np.asarray(batch["obs"], dtype=np.float64), e)
    R = x.shape[0]
    z1, h1, z2, h2 = _forward_torso(x, W1, b1, W2, b2, e)
    logits = h2 @ Wa.T + ba
    a = np.asarray(batch["actions"], dtype=np.int64)
    logp_all = _log_softmax(logits)
    prob = np.exp(logp_all)
    logp = logp_all[np.arange(R), a]
    rho = np.exp(logp - np.asarray(batch["logp_old"], dtype=np.float64))
    ahat = normalise(batch["adv"])
    # surrogate: the unclipped branch carries the gradient unless the clipped one is the smaller
    inside = (rho >= 1.0 - hp.clip_eps) & (rho <= 1.0 + hp.clip_eps)
    unclipped_is_min = rho * ahat < np.clip(rho, 1.0 - hp.clip_eps, 1.0 + hp.clip_eps) * ahat
    d_logp = -(rho * ahat) * (inside | unclipped_is_min) / R             # dL/dlogp(a)
    onehot = np.zeros_like(logits)
    onehot[np.arange(R), a] = 1.0
    H = -(prob * logp_all).sum(axis=1, keepdims=True)
    d_logits = d_logp[:, None] * (onehot - prob)                           # dlogp(a)/dz_k = [k = a] - p_k
    d_logits += hp.ent_coef / R * prob * (logp_all + H)                    # -c_ent dHbar/dz_k, dH/dz_k = -p_k (log p_k + H)

    def value_grad(values, v_old, ret):
        n = values.shape[0]
        u, uc = values - ret, v_old + np.clip(values - v_old, -hp.clip_eps, hp.clip_eps) - ret
        in_range = np.abs(values - v_old) <= hp.clip_eps
        d = np.where(in_range | (u * u > uc * uc), u, 0.0)                 # the clipped term, when larger, is constant in V
        return hp.vf_coef * d / n

    v_old = np.asarray(batch["value_old"], dtype=np.float64)
    ret = np.asarray(batch["ret"], dtype=np.float64)
    grads = []
    dba = d_logits.sum(axis=0)          # the unrounded derivatives
    d_logits = _r(d_logits, e)          # as operands of the two products below
    dWa = d_logits.T @ h2
    dh2 = d_logits @ Wa
    if net_kind == 0:
        (Wv, bv) = p[3]
        Wv = _r(Wv, e)
        values = (h2 @ Wv.T + bv)[:, 0]
        dv = value_grad(values, v_old, ret)
        dbv = np.array([dv.sum()])
        dv = _r(dv, e)
        dWv = dv[None, :] @ h2
        dh2 = dh2 + dv[:, None] * Wv
        dW1, db1, dW2, db2 = _backward_torso(x, z1, h1, z2, h2, dh2, W2, e)
        grads = [dW1, db1, dW2, db2, dWa, dba, dWv, dbv]
    else:
        dW1, db1, dW2, db2 = _backward_torso(x, z1, h1, z2, h2, dh2, W2, e)
        (C1, c1), (C2, c2), (Cv, cv) = p[3], p[4], p[5]
        C1, C2, Cv = _r(C1, e), _r(C2, e), _r(Cv, e)
        xj = _r(np.asarray(batch["joint_obs"], dtype=np.float64), e)
        y1, g1, y2, g2 = _forward_torso(xj, C1, c1, C2, c2, e)
        values = (g2 @ Cv.T + cv)[:, 0]
        dv = value_grad(values, v_old, ret)
        dcv = np.array([dv.sum()])
        dv = _r(dv, e)
        dCv = dv[None, :] @ g2
        dC1, dc1, dC2, dc2 = _backward_torso(xj, y1, g1, y2, g2, dv[:, None] * Cv, C2, e)
        grads = [dW1, db1, dW2, db2, dWa, dba, dC1, dc1, dC2, dc2, dCv, dcv]
    return np.concatenate([g.ravel() for g in grads])


def clip_by_global_norm(grad, max_norm: float):
    """The gradient scaled so that its 2-norm is at most `max_norm` (unchanged when already below)."""
    grad = np.asarray(grad, dtype=np.float64)
    norm = np.sqrt((grad * grad).sum())
    return grad * (max_norm / max(norm, max_norm)), norm


def adam_step(params, grad, m, v, step: int, hp: Hyper = Hyper()):
    """One Adam update (step counts from 1); returns (params, m, v), all float64."""
    g, _ = clip_by_global_norm(grad, hp.max_grad_norm)
    m = hp.beta1 * m + (1.0 - hp.beta1) * g
    v = hp.beta2 * v + (1.0 - hp.beta2) * g * g
    m_hat = m / (1.0 - hp.beta1 ** step)
    v_hat = v / (1.0 - hp.beta2 ** step)
    return np.asarray(params, dtype=np.float64) - hp.lr * m_hat / (np.sqrt(v_hat) + hp.adam_eps), m, v


def batch_from_rollout(obs, actions, logp, values, adv, ret, net_kind: int):
    """A minibatch holding every row of a stored trajectory (time-major arrays as the rollout writes
    them: obs [T][E][N][D], actions/logp/adv/ret [T][E][N], values [T+1][E][N])."""
    T, E, N, D = obs.shape
    b = {"obs": obs.reshape(T * E * N, D), "actions": actions.reshape(-1), "logp_old": logp.reshape(-1),
         "adv": adv.reshape(-1)}
    if net_kind == 0:
        b["value_old"] = values[:T].reshape(-1)
        b["ret"] = ret.reshape(-1)
    else:
        b["joint_obs"] = obs.reshape(T * E, N * D)
        b["value_old"] = values[:T, :, 0].reshape(-1)
        b["ret"] = ret[:, :, 0].reshape(-1)
    return b
