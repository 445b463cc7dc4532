#!/usr/bin/env python
"""Benchmark of the fused rollout + GAE path (one JSON line on stdout).

A "step" is one pass of the whole path over one batch: mava_rollout_run (T environment steps of
E environments, MLP forward, sampling, auto-reset, trajectory stores) followed by mava_gae.
`value` = env-agent-steps per second = E*N*T / (device time of the step), inputs resident in HBM.
`e2e` = the same through mava_rollout_collect_host (parameters copied from pinned host memory
and the whole trajectory copied back inside the timed region).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 0..4] [--impl reference]

With N > 1 (torchrun) every rank rolls its own shard of N*E environments (first_env = rank*E);
there is no data-path collective, only the barrier and the max-over-ranks of the timings.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2107_01460_b200 import workloads as wl  # noqa: E402

METRIC = "env_agent_steps_per_s"
UNIT = "env-agent-steps/s"
DEFAULT_WORKLOAD = 4  # the largest workload that fits one GPU
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# ---- algorithmic work of one agent row (one agent, one step) ---------------------------------

def bytes_per_row(w) -> float:
    """Bytes the path must write per agent row: obs (4D) + action, logp, value, reward (4 each)
    + the env's done byte shared by its N agents.  Nothing has to be read from HBM."""
    return 4.0 * wl.obs_dim(w) + 16.0 + 1.0 / w["n_agents"]


def flops_per_row(w) -> float:
    """2 * multiply-accumulates of the unpadded network, per agent row."""
    D, H, N = wl.obs_dim(w), w["hidden"], w["n_agents"]
    if w["net_kind"] == 2:  # recurrent: embedding, the cell's two [3H][H] matrices, the heads
        return 2.0 * (D * H + 6 * H * H + 7 * H)
    macs = D * H + H * H + 6 * H
    if w["net_kind"] == 0:
        macs += H
    else:
        macs += (N * D * H + H * H + H) / N  # one critic forward per environment
    return 2.0 * macs


def gae_bytes_per_element(w) -> float:
    """value + reward read, advantage + return written, the done byte shared by N agents."""
    return 16.0 + 1.0 / w["n_agents"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


def ncu_traffic(w, precision_name):
    """DRAM bytes (read + write) of one launch of the rollout kernel on workload `w`, from the table of ncu captures
    kept with the profiler summaries; None when there is no capture of this workload or when the kernel's sources
    have changed since it was taken.  A capture of fewer environments is scaled by the environment count (traffic is
    trajectory writes, proportional to the rows)."""
    import hashlib

    path = os.path.join(ROOT, "profiles", "ncu_dram_traffic.txt")
    if not os.path.exists(path):
        return None, None
    csrc = os.path.join(ROOT, "paper_2107_01460_b200", "csrc")
    digest = hashlib.sha256()
    for name in ("rollout_tc.cu", "rollout_tc_small.cuh", "env.cuh", "tc_common.cuh", "common.cuh"):
        with open(os.path.join(csrc, name), "rb") as fh:
            digest.update(fh.read())
    digest = digest.hexdigest()[:16]
    with open(path) as fh:
        for line in fh:
            parts = line.split()
            if len(parts) < 6 or parts[0].startswith("#"):
                continue
            name, prec, envs, read_b, write_b, src = parts[:6]
            if name == w["name"] and prec == precision_name:
                if src != digest:
                    return None, "the rollout kernel's sources changed after the ncu capture"
                scale = w["n_envs"] / float(envs)
                note = "ncu dram__bytes_read.sum + dram__bytes_write.sum, one launch"
                if scale != 1.0:
                    note += f", captured at {envs} environments and scaled by {scale:g}"
                return (float(read_b) + float(write_b)) * scale, note
    return None, None


# ---- clock sampling -----------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100", "-i",
                 str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---- CPU oracle timing (cpu_baseline leg and --impl reference) ------------------------------

def oracle_sample_run(w, params, n_sample_envs: int, n_threads: int):
    """Times the oracle, as it stands, on the first `n_sample_envs` environments for the full T
    (rollout + GAE), environments split over `n_threads` host threads.  Returns (rows, seconds)."""
    import oracle  # the one place outside tests/smoke that may execute the oracle

    ocfg = oracle.make_config(w)
    T, N = w["T"], w["n_agents"]
    chunks = [c for c in np.array_split(np.arange(n_sample_envs, dtype=np.int32), n_threads) if c.size]
    results = [None] * len(chunks)

    def work(i):
        if w["net_kind"] == 2:
            ro, _ = oracle.rollout_rec(ocfg, w["seed"], params, T, chunks[i], want_obs=True)
        else:
            ro = oracle.rollout(ocfg, w["seed"], params, T, chunks[i], want_obs=True)
        adv, ret = oracle.gae(ro.values.astype(np.float32), ro.rewards, ro.dones, wl.GAMMA, wl.LAMBDA)
        results[i] = adv.shape

    t0 = time.perf_counter()
    threads = [threading.Thread(target=work, args=(i,)) for i in range(len(chunks))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    dt = time.perf_counter() - t0
    return n_sample_envs * N * T, dt, len(chunks)


def sample_envs_for(w, seconds_target: float, cores: int) -> int:
    """Sample size giving roughly `seconds_target` of oracle work (about 2.5e8 MAC/s per core)."""
    rows_per_env = w["n_agents"] * w["T"]
    rate = 2.5e8 * cores / (flops_per_row(w) / 2.0)  # rows per second
    n = int(max(cores, min(w["n_envs"], seconds_target * rate / rows_per_env)))
    return n


def oracle_baseline(w, seconds_each: float):
    """The oracle as it stands on a bounded sample of workload `w` (the first min(E, 256) environments for the full T,
    rollout + GAE; env-agent-steps/s is per row, so the figure does not depend on E): once on one thread with a
    smaller sample, once with the environments split over all host cores; each repeated until `seconds_each` of wall
    time have gone by."""
    params = wl.make_params(w)
    cores = os.cpu_count() or 1
    n_multi = min(w["n_envs"], 256)
    n_single = max(1, min(n_multi, sample_envs_for(w, seconds_each / 2.0, 1)))
    out = {}
    for label, n_env, n_thr in (("single_thread", n_single, 1), ("all_cores", n_multi, cores)):
        rows, secs, passes, used = 0, 0.0, 0, n_thr
        while secs < seconds_each and passes < 4096:
            r_, s_, used = oracle_sample_run(w, params, n_env, n_thr)
            rows += r_; secs += s_; passes += 1
        out[label] = {"value": rows / secs, "unit": UNIT, "cores": used, "kind": "oracle",
                      "sample": f"first {n_env} of {w['n_envs']} envs x full T={w['T']} (rollout + GAE), {passes} pass(es), "
                                f"{secs:.1f} s wall"}
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    w = wl.workload(args.workload)
    params = wl.make_params(w)
    cores = os.cpu_count() or 1
    n_sample = sample_envs_for(w, 3.0, cores)
    for _ in range(args.warmup):
        oracle_sample_run(w, params, max(cores, n_sample // 8), cores)
    total_rows, total_s, used = 0, 0.0, cores
    for _ in range(args.steps):
        rows, dt, used = oracle_sample_run(w, params, n_sample, cores)
        total_rows += rows
        total_s += dt
    value = total_rows / total_s
    sample = f"first {n_sample} of {w['n_envs']} envs x full T={w['T']} per step (rollout + GAE)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total_s / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w["name"], "n_envs_per_gpu": w["n_envs"], "T": w["T"], "n_agents": w["n_agents"],
                   "hidden": w["hidden"], "obs_dim": wl.obs_dim(w), "global_envs": w["n_envs"],
                   "parallelism": "env-shards x1", "l2": "host run: no device cache to flush"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ---- GPU arm ------------------------------------------------------------------------------------

def pick_precision(binding, w):
    """The workload's stated arithmetic if the library has it compiled, else the fp32 path."""
    want = binding.MAVA_PRECISION_BF16 if w["precision"] == "bf16" else binding.MAVA_PRECISION_FP32
    if want == binding.MAVA_PRECISION_BF16:
        try:
            binding.Rollout(binding.make_config(w, precision=want, n_envs=2, max_T=1)).close()
        except binding.MavaError:
            want = binding.MAVA_PRECISION_FP32
    return want


def time_workload(torch, binding, w, precision, steps, warmup, first_env=0, flush=None):
    """Device timing of `steps` steps; returns per-step lists (ms) of rollout and GAE times."""
    cfg = binding.make_config(w, precision=precision, first_env=first_env)
    ro = binding.Rollout(cfg)
    params = torch.from_numpy(wl.make_params(w)).cuda()
    T = w["T"]
    t_roll, t_gae = [], []
    launches0 = 0
    for i in range(warmup + steps):
        if i == warmup:
            launches0 = ro.launch_count()
        if flush is not None:
            flush.add_(1.0)  # writes a buffer larger than L2 between steps (outside the events)
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        ro.run(params, T)
        e1.record()
        ro.gae(wl.GAMMA, wl.LAMBDA)
        e2.record()
        e2.synchronize()
        if i >= warmup:
            t_roll.append(e0.elapsed_time(e1))
            t_gae.append(e1.elapsed_time(e2))
    assert ro.status() == binding.MAVA_OK
    launches = ro.launch_count() - launches0
    return ro, params, t_roll, t_gae, launches


def time_evaluate(torch, ro, params, w, steps, warmup, flush):
    """Device timing of greedy evaluation blocks of the workload's T steps (ms per block)."""
    times = []
    for i in range(warmup + steps):
        flush.add_(1.0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ro.evaluate(params, w["T"], greedy=True)
        e1.record()
        e1.synchronize()
        if i >= warmup:
            times.append(e0.elapsed_time(e1))
    return sum(times) / len(times)


def time_update(torch, binding, ro, params, w, steps, warmup, flush):
    """Device timing of the update block on the rows of one rollout: PPO loss + gradient, then one Adam step (ms);
    also names the arithmetic path the handle's precision selects."""
    ro.run(params, w["T"])
    ro.gae(wl.GAMMA, wl.LAMBDA)
    p = params.clone()
    m, v = torch.zeros_like(p), torch.zeros_like(p)
    times = []
    for i in range(warmup + steps):
        flush.add_(1.0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        _, grad = ro.ppo_grad(p)
        ro.adam_step(p, grad, m, v, i + 1)
        e1.record()
        e1.synchronize()
        if i >= warmup:
            times.append(e0.elapsed_time(e1))
    path = "fp32 SIMT"
    if binding.update_on_tensor_cores(ro.cfg):
        path = "bf16 tcgen05"
    return sum(times) / len(times), path


def time_e2e(torch, binding, ro, w, steps, warmup):
    T, E, N, D = w["T"], w["n_envs"], w["n_agents"], wl.obs_dim(w)
    pin = lambda shape, dt: torch.empty(shape, dtype=dt).pin_memory()  # noqa: E731
    out = {"obs": pin((T, E, N, D), torch.float32), "actions": pin((T, E, N), torch.int32),
           "logp": pin((T, E, N), torch.float32), "values": pin((T + 1, E, N), torch.float32),
           "rewards": pin((T, E, N), torch.float32), "dones": pin((T, E), torch.uint8),
           "adv": pin((T, E, N), torch.float32), "ret": pin((T, E, N), torch.float32)}
    params_host = torch.from_numpy(wl.make_params(w)).pin_memory()
    d2h = sum(t.numel() * t.element_size() for t in out.values())
    h2d = params_host.numel() * 4
    times = []
    for i in range(warmup + steps):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ro.collect_host(params_host, T, wl.GAMMA, wl.LAMBDA, out)  # synchronous
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    return sum(times) / len(times), h2d, d2h


def rollout_roofline(w, rows, roll_ms, peaks, precision):
    """The rollout launch against the slower of its two bounds.  A kernel timed alone between L2 flushes is measured
    against the burst tensor peak; the fraction of the sustained (power-capped, seconds-long) peak is given beside it."""
    t_hbm = rows * bytes_per_row(w) / (peaks["hbm_gbs"] * 1e9)
    t_tensor = rows * flops_per_row(w) / (peaks["bf16_tflops"] * 1e12)
    if t_hbm >= t_tensor:
        ach = rows * bytes_per_row(w) / (roll_ms * 1e-3) / 1e9
        r = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"]}
    else:
        ach = rows * flops_per_row(w) / (roll_ms * 1e-3) / 1e12
        r = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
             "frac": ach / peaks["bf16_tflops"], "peak_kind": "burst (kernel timed alone)",
             "frac_of_sustained_peak": ach / peaks["bf16_tflops_sustained"],
             "sustained_peak": peaks["bf16_tflops_sustained"]}
    r["kernel"] = "rollout (fused env step + MLP + sampler), %s" % ("bf16 tcgen05" if precision else "fp32 SIMT")
    r["traffic"], r["traffic_note"] = ncu_traffic(w, "bf16" if precision else "fp32")
    r["peak_source"] = "of " + peaks["source"]
    r["kernel_ms"] = roll_ms
    r["algorithmic_bytes"] = rows * bytes_per_row(w)
    r["algorithmic_flops"] = rows * flops_per_row(w)
    return r


def update_report(w, rows, upd_ms, upd_path, peaks):
    """Update block: forward and the two backward products of every layer = 3 x the forward FLOPs, against the bf16
    tensor peak (the block's products are GEMMs over the rollout's rows)."""
    ach = 3 * rows * flops_per_row(w) / (upd_ms * 1e-3) / 1e12
    return {"value": rows / (upd_ms * 1e-3), "unit": "rows/s", "ms": upd_ms, "bound": "tensor", "achieved": ach,
            "peak": peaks["bf16_tflops"], "unit_roofline": "TFLOP/s", "frac": ach / peaks["bf16_tflops"],
            "path": upd_path + " (mava_ppo_grad + mava_adam_step), all rows of the rollout as one minibatch"}


def run_gpu(args):
    import torch

    from paper_2107_01460_b200 import binding, build

    build.build()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks = load_peaks()
    w = wl.workload(args.workload)
    precision = pick_precision(binding, w)
    E, N, T = w["n_envs"], w["n_agents"], w["T"]
    rows = E * N * T
    flush = torch.zeros(64 * 1024 * 1024, dtype=torch.float32, device="cuda")  # 256 MiB > 126 MB L2

    sampler = ClockSampler(local_rank)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    ro, params, t_roll, t_gae, launches = time_workload(torch, binding, w, precision, args.steps, args.warmup,
                                                        first_env=wl.shard_first_env(E, rank), flush=flush)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if dist is not None:
        dist.barrier()
    step_ms = (sum(t_roll) + sum(t_gae)) / args.steps
    e2e_s, h2d, d2h = time_e2e(torch, binding, ro, w, max(3, args.steps // 4), 2)
    eval_ms = time_evaluate(torch, ro, params, w, max(3, args.steps // 4), 3, flush)  # rank-local, reported by rank 0
    upd_ms, upd_path = time_update(torch, binding, ro, params, w, max(3, args.steps // 4), 3, flush) if rank == 0 else (0.0, "")
    if dist is not None:
        t = torch.tensor([step_ms, e2e_s], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        step_ms, e2e_s = float(t[0]), float(t[1])
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    roll_ms = sum(t_roll) / len(t_roll)
    gae_ms = sum(t_gae) / len(t_gae)
    roofline = rollout_roofline(w, rows, roll_ms, peaks, precision)
    gae_ach = rows * gae_bytes_per_element(w) / (gae_ms * 1e-3) / 1e9
    gae = {"elements_per_s": rows / (gae_ms * 1e-3), "kernel_ms": gae_ms, "bound": "hbm", "achieved": gae_ach,
           "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gae_ach / peaks["hbm_gbs"]}
    update = update_report(w, rows, upd_ms, upd_path, peaks)
    del ro, params
    torch.cuda.empty_cache()

    # every workload of the table, briefly: device times, roofline fractions, and the oracle beside each
    sweep = []
    if not args.no_sweep and world == 1:
        for idx in range(len(wl.WORKLOAD_NAMES)):
            wi = wl.workload(idx)
            pi = pick_precision(binding, wi)
            r_i, p_i, tr, tg, _ = time_workload(torch, binding, wi, pi, 5, 3, flush=flush)
            recurrent = wi["net_kind"] == 2  # the recurrent policy has a rollout and GAE, no update block
            tu_ms, tu_path = (None, None) if recurrent else time_update(torch, binding, r_i, p_i, wi, 2, 1, flush)
            del r_i, p_i
            torch.cuda.empty_cache()
            ri = wi["n_envs"] * wi["n_agents"] * wi["T"]
            tr_ms, tg_ms = sum(tr) / len(tr), sum(tg) / len(tg)
            rf = rollout_roofline(wi, ri, tr_ms, peaks, pi)
            entry = {"workload": wi["name"], "precision": "bf16" if pi else "fp32", "rollout_ms": tr_ms,
                     "gae_ms": tg_ms, "env_agent_steps_per_s": ri / ((tr_ms + tg_ms) * 1e-3),
                     "rollout_roofline_bound": rf["bound"], "rollout_roofline_frac": rf["frac"],
                     "rollout_roofline_frac_of_sustained_peak": rf.get("frac_of_sustained_peak"),
                     "rollout_us_per_env_step": 1e3 * tr_ms / wi["T"],
                     "gae_elements_per_s": ri / (tg_ms * 1e-3),
                     "gae_hbm_frac": ri * gae_bytes_per_element(wi) / (tg_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     "update_ms": tu_ms, "update_path": tu_path}
            if tu_ms is not None:
                entry["update_rows_per_s"] = ri / (tu_ms * 1e-3)
                entry["update_tensor_frac"] = 3 * ri * flops_per_row(wi) / (tu_ms * 1e-3) / 1e12 / peaks["bf16_tflops"]
            if not args.no_oracle:
                entry["cpu_baseline"] = oracle_baseline(wi, args.oracle_seconds)
            sweep.append(entry)

    # CPU baseline of the headline workload: the oracle on a bounded sample of it
    if sweep and "cpu_baseline" in sweep[args.workload]:
        cpu = dict(sweep[args.workload]["cpu_baseline"]["all_cores"])
        cpu["single_thread"] = sweep[args.workload]["cpu_baseline"]["single_thread"]
    else:
        both = oracle_baseline(w, args.oracle_seconds)
        cpu = dict(both["all_cores"])
        cpu["single_thread"] = both["single_thread"]

    line = {
        "metric": METRIC, "value": world * rows / (step_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if precision else "f32", "data": "synthetic",
        "config": {"workload": w["name"], "n_envs_per_gpu": E, "T": T, "n_agents": N, "hidden": w["hidden"],
                   "obs_dim": wl.obs_dim(w), "global_envs": world * E, "parallelism": f"env-shards x{world}",
                   "l2": "256 MiB buffer rewritten between steps (outside the per-step events)"},
        "clocks": clocks,
        "e2e": {"value": world * rows / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": launches,
        "roofline": roofline,
        "gae": gae,
        "evaluate": {"value": rows / (eval_ms * 1e-3), "unit": UNIT, "ms_per_block": eval_ms,
                     "block": f"greedy, T={T} steps, no trajectory stored (mava_rollout_evaluate), one GPU"},
        "update": update,
        "cpu_baseline": cpu,
        "workloads": sweep,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=DEFAULT_WORKLOAD, help="index 0..4 of the workload table")
    ap.add_argument("--no-sweep", action="store_true", help="skip the brief timing of the other workloads")
    ap.add_argument("--no-oracle", action="store_true", help="skip the oracle timing beside every workload of the sweep")
    ap.add_argument("--oracle-seconds", type=float, default=8.0, help="wall time of each oracle timing (per workload: one thread, all cores)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    return run_reference(args) if args.impl == "reference" else run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
