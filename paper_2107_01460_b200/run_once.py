"""Run one workload a few times through the C ABI and print the device times (for profilers).

    python -m paper_2107_01460_b200.run_once --workload 2 [--precision bf16|fp32] [--repeats 3] [--envs E] [--update]
"""
from __future__ import annotations

import argparse

import torch

from . import binding, build, workloads as wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", type=int, default=1)
    ap.add_argument("--precision", default=None, choices=[None, "bf16", "fp32"])
    ap.add_argument("--repeats", type=int, default=3)
    ap.add_argument("--envs", type=int, default=None, help="override the number of environments")
    ap.add_argument("--update", action="store_true", help="also run the update block (PPO gradient + Adam step) on the rows")
    args = ap.parse_args()
    build.build()
    w = wl.workload(args.workload)
    prec = {None: None, "bf16": binding.MAVA_PRECISION_BF16, "fp32": binding.MAVA_PRECISION_FP32}[args.precision]
    cfg = binding.make_config(w, precision=prec, n_envs=args.envs)
    ro = binding.Rollout(cfg)
    params = torch.from_numpy(wl.make_params(w)).cuda()
    rows = cfg.n_envs * cfg.n_agents * w["T"]
    for i in range(args.repeats):
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record(); ro.run(params, w["T"]); e1.record(); ro.gae(wl.GAMMA, wl.LAMBDA); e2.record()
        e2.synchronize()
        if args.update:
            if i == 0:
                m, v = torch.zeros_like(params), torch.zeros_like(params)
            e3 = torch.cuda.Event(enable_timing=True)
            terms, grad = ro.ppo_grad(params)
            ro.adam_step(params.clone(), grad, m, v, i + 1)
            e3.record(); e3.synchronize()
            print(f"run {i}: update {e2.elapsed_time(e3):.4f} ms, loss {terms[0].item():.6f}")
        print(f"run {i}: rollout {e0.elapsed_time(e1):.4f} ms, gae {e1.elapsed_time(e2):.4f} ms, "
              f"{rows / (e0.elapsed_time(e2) * 1e-3):.4g} env-agent-steps/s")
    assert ro.status() == binding.MAVA_OK
    ro.close()


if __name__ == "__main__":
    main()
