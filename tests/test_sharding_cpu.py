"""World-size-2 gloo test of the multi-GPU host logic: environments shard across ranks with no
collective on the data path (Philox is keyed on global environment indices), and the benchmark's
max-over-ranks timing reduction works."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2107_01460_b200 import workloads as wl


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
