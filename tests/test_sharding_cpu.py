"""World-size-2 gloo test of the multi-GPU host logic: environments shard across ranks with no
collective on the data path (Philox is keyed on global environment indices), and the benchmark's
max-over-ranks timing reduction works; the update block's one exchange, the gradient mean, is the
all-reduce of `train.average_gradients`."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from oracle import ppo
from paper_2107_01460_b200 import train, workloads as wl


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.workload(0)
    per_rank = 5
    first = wl.shard_first_env(per_rank, rank)
    ids = np.arange(first, first + per_rank, dtype=np.int32)
    ro = oracle.rollout(oracle.make_config(w), w["seed"], wl.make_params(w), 12, ids)
    np.save(os.path.join(out_dir, f"obs{rank}.npy"), ro.obs)
    np.save(os.path.join(out_dir, f"act{rank}.npy"), ro.actions)
    # the warehouse family (its replacement requests are keyed on global indices too) and the recurrent policy
    ww = wl.workload("wh2_10x10_3r3s_h128_collisions_end")
    wh = oracle.rollout(oracle.make_config(ww), ww["seed"], wl.make_params(ww), 30, ids)
    np.save(os.path.join(out_dir, f"wh{rank}.npy"), np.concatenate([wh.obs.reshape(30, per_rank, -1), wh.rewards], axis=2))
    wr = wl.workload("rec0_tiny_8x8_2p2f_gru64")
    rec, hid = oracle.rollout_rec(oracle.make_config(wr), wr["seed"], wl.make_params(wr), 12, ids)
    np.save(os.path.join(out_dir, f"rec{rank}.npy"), rec.logits)
    t = torch.tensor([1.0 + rank, 10.0 - rank], dtype=torch.float64)  # (step ms, e2e s) of this rank
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert t.tolist() == [float(world), 10.0]
    dist.barrier()
    dist.destroy_process_group()


def test_env_shards_reproduce_the_unsharded_batch(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    w = wl.workload(0)
    whole = oracle.rollout(oracle.make_config(w), w["seed"], wl.make_params(w), 12, np.arange(10, dtype=np.int32))
    obs = np.concatenate([np.load(tmp_path / f"obs{r}.npy") for r in range(world)], axis=1)
    act = np.concatenate([np.load(tmp_path / f"act{r}.npy") for r in range(world)], axis=1)
    assert np.array_equal(obs, whole.obs) and np.array_equal(act, whole.actions)
    ids = np.arange(10, dtype=np.int32)
    ww = wl.workload("wh2_10x10_3r3s_h128_collisions_end")
    wh = oracle.rollout(oracle.make_config(ww), ww["seed"], wl.make_params(ww), 30, ids)
    got = np.concatenate([np.load(tmp_path / f"wh{r}.npy") for r in range(world)], axis=1)
    assert np.array_equal(got, np.concatenate([wh.obs.reshape(30, 10, -1), wh.rewards], axis=2))
    wr = wl.workload("rec0_tiny_8x8_2p2f_gru64")
    rec, _ = oracle.rollout_rec(oracle.make_config(wr), wr["seed"], wl.make_params(wr), 12, ids)
    assert np.array_equal(np.concatenate([np.load(tmp_path / f"rec{r}.npy") for r in range(world)], axis=1), rec.logits)


def _shard_gradient(rank, per_rank, T):
    """PPO gradient (float64 oracle) of one rank's shard of environments, as the update kernel forms it: over the
    shard's own rows, advantages normalised over those rows."""
    w = wl.workload(0)
    params = wl.make_params(w, bias_scale=0.1)
    first = wl.shard_first_env(per_rank, rank)
    ro = oracle.rollout(oracle.make_config(w), w["seed"], params, T, np.arange(first, first + per_rank, dtype=np.int32))
    adv, ret = oracle.gae(ro.values, ro.rewards, ro.dones, wl.GAMMA, wl.LAMBDA)
    shapes = ppo.layer_shapes(wl.obs_dim(w), w["hidden"], w["n_agents"], w["net_kind"])
    batch = ppo.batch_from_rollout(ro.obs, ro.own_actions, ro.logp, ro.values, adv, ret, w["net_kind"])
    p64 = params.astype(np.float64) * 1.05  # a little away from the rollout's parameters, so that ratios leave 1
    return ppo.ppo_grad(p64, shapes, w["net_kind"], batch)


def _grad_worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.from_numpy(_shard_gradient(rank, 4, 10))
    train.average_gradients(g)
    np.save(os.path.join(out_dir, f"avg{rank}.npy"), g.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_gradient_mean_across_ranks(tmp_path):
    world = 2
    mp.spawn(_grad_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    want = sum(_shard_gradient(r, 4, 10) for r in range(world)) / world
    for r in range(world):
        got = np.load(tmp_path / f"avg{r}.npy")
        assert np.max(np.abs(got - want)) <= 1e-15 * max(1.0, np.max(np.abs(want)))
    # without a process group the call leaves the gradient alone
    g = torch.ones(5, dtype=torch.float64)
    assert torch.equal(train.average_gradients(g.clone()), g)
