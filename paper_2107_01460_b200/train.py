"""The whole on-device loop the report describes (Section 2, Figure 2): roll out, estimate advantages, update,
repeat, with evaluation blocks in between -- every step of the method is a call into the C ABI; Python drives the
loop, draws the minibatch permutations, averages the printed returns and, across ranks, sums the gradient.

    python -m paper_2107_01460_b200.train [--workload 1] [--envs 1024] [--steps 64] [--iters 200] [--epochs 4]
                                          [--lr 1e-3] [--eval-every 25] [--minibatches 1]

Each iteration: mava_rollout_run (T steps of every environment, continuing where the last one stopped), mava_gae,
then `epochs` passes of mava_ppo_grad + mava_adam_step over the rows of that rollout, as one minibatch or, with
--minibatches k, as k minibatches of environments drawn from a fresh permutation per pass.  Every
`eval-every` iterations a second handle with the same shape runs a greedy evaluation block from fresh episodes and
the mean return of the episodes that ended is printed (1.0 = every food item collected).

Under torchrun (one process per GPU) every rank rolls out its own shard of the environments (`first_env` = rank x
envs, so the shards are the environments of one large batch) and the ranks exchange one thing per update: the
gradient, averaged with an NCCL all-reduce (the report's `pmean`, Section 2).  Parameters and optimiser state start
equal and see the same averaged gradient, so they stay equal without being sent.
"""
from __future__ import annotations

import argparse

import torch

from . import binding, build, workloads as wl


def mean_return(ev: "binding.Rollout", params, T: int, seed: int) -> float:
    """Mean return of the episodes that end inside a greedy block of T steps from fresh episodes."""
    ev.reset(seed)
    count, ret, _, _ = ev.evaluate(params, T, greedy=True)
    n = int(count.sum().item())
    return float(ret.sum().item()) / n if n else float("nan")


def average_gradients(grad):
    """In place: the mean of `grad` over the ranks of the default process group (a no-op without one)."""
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(grad, op=dist.ReduceOp.SUM)
        grad /= dist.get_world_size()
    return grad


def train(workload: int = 1, n_envs: int = 1024, T: int = 64, iters: int = 200, epochs: int = 4, lr: float = 1e-3,
          eval_every: int = 25, precision: int | None = None, log=print, rank: int = 0, minibatches: int = 1):
    """Runs the loop and returns the list of (iteration, mean greedy return) it evaluated."""
    build.build()
    w = wl.workload(workload)
    cfg = binding.make_config(w, precision=precision, n_envs=n_envs, max_T=T, first_env=wl.shard_first_env(n_envs, rank))
    device = f"cuda:{torch.cuda.current_device()}"
    ro = binding.Rollout(cfg, device=device)
    cap = w["episode_cap"]
    ev = binding.Rollout(binding.make_config(w, precision=precision, n_envs=n_envs, max_T=2 * cap), device=device, with_gae=False)
    params = torch.from_numpy(wl.make_params(w)).cuda()
    m, v = torch.zeros_like(params), torch.zeros_like(params)
    hp = binding.ppo_defaults()
    hp.lr = lr
    history, step = [], 0
    shuffle = torch.Generator(device="cuda").manual_seed(1234 + rank)
    for it in range(iters + 1):
        if it % eval_every == 0 or it == iters:
            r = mean_return(ev, params, 2 * cap, seed=10_000 + it)
            history.append((it, r))
            log(f"iteration {it:4d}: mean greedy return {r:.4f}")
        if it == iters:
            break
        ro.run(params, T)
        ro.gae(wl.GAMMA, wl.LAMBDA)
        import torch.distributed as dist

        if not (dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1):
            # one process: the passes and minibatches of the iteration in one library call; the shuffling (a fresh
            # permutation per pass, seeded, same on every run) is drawn here and handed over
            perm = torch.stack([torch.randperm(n_envs, generator=shuffle, device="cuda") if minibatches > 1
                                else torch.arange(n_envs, device="cuda") for _ in range(epochs)]).to(torch.int32).contiguous()
            ro.ppo_update(params, m, v, perm, max(1, minibatches), step + 1, hp)
            step += epochs * max(1, minibatches)
            continue
        for _ in range(epochs):
            # several ranks: the gradient is averaged between the gradient call and the optimiser call
            pieces = [None] if minibatches <= 1 else torch.randperm(n_envs, generator=shuffle, device="cuda").to(torch.int32).chunk(minibatches)
            for ids in pieces:
                step += 1
                terms, grad = ro.ppo_grad(params, hp, env_ids=None if ids is None else ids.contiguous())
                average_gradients(grad)
                ro.adam_step(params, grad, m, v, step, hp)
    assert ro.status() == binding.MAVA_OK and ev.status() == binding.MAVA_OK
    ro.close()
    ev.close()
    return history


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", type=int, default=1)
    ap.add_argument("--envs", type=int, default=1024)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--iters", type=int, default=200)
    ap.add_argument("--epochs", type=int, default=4)
    ap.add_argument("--lr", type=float, default=1e-3)
    ap.add_argument("--eval-every", type=int, default=25)
    ap.add_argument("--minibatches", type=int, default=1, help="pieces of a shuffled epoch (environments per piece = envs / this)")
    args = ap.parse_args()
    import os

    rank = 0
    if "RANK" in os.environ and int(os.environ.get("WORLD_SIZE", "1")) > 1:
        import torch.distributed as dist

        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
        dist.init_process_group("nccl")
        rank = dist.get_rank()
    train(args.workload, args.envs, args.steps, args.iters, args.epochs, args.lr, args.eval_every,
          log=print if rank == 0 else (lambda *_: None), rank=rank, minibatches=args.minibatches)
    if rank or "RANK" in os.environ:
        import torch.distributed as dist

        if dist.is_initialized():
            dist.destroy_process_group()


if __name__ == "__main__":
    main()
