"""The multi-GPU path on CPU: two gloo ranks, each simulating its shard (the
oracle stands in for the device), must reproduce the one-process batch exactly,
and the cross-rank reductions (max time, summed counters) must be right."""
import os
import socket

import numpy as np
import pytest

import oracle
from paper_2603_12145_b200 import sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, n_per_rank, T, seed, out_dir):
    import torch
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        base, n = sharding.shard(rank, world, n_per_rank)
        o = oracle.OraclePong(n, seed, env_id_base=base)
        obs, reward, done = o.rollout(T, 1)
        dist.barrier()
        tmax = sharding.max_over_ranks(10.0 + rank)
        total = sharding.sum_stats(o.episode_stats())
        np.savez(os.path.join(out_dir, "rank%d.npz" % rank), obs=obs, reward=reward, done=done,
                 tmax=tmax, total=np.array(total), local=np.array(o.episode_stats()))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_single_process_batch(tmp_path):
    import torch.multiprocessing as mp
    world, n_per_rank, T, seed = 2, 24, 3000, 5
    port = _free_port()
    mp.spawn(_rank_main, args=(world, port, n_per_rank, T, seed, str(tmp_path)), nprocs=world,
             join=True)
    whole = oracle.OraclePong(world * n_per_rank, seed)
    obs, reward, done = whole.rollout(T, 1)
    parts = [np.load(os.path.join(str(tmp_path), "rank%d.npz" % r)) for r in range(world)]
    for r, p in enumerate(parts):
        lo, hi = r * n_per_rank, (r + 1) * n_per_rank
        assert p["obs"].tobytes() == np.ascontiguousarray(obs[:, lo:hi]).tobytes()
        assert p["reward"].tobytes() == np.ascontiguousarray(reward[:, lo:hi]).tobytes()
        assert p["done"].tobytes() == np.ascontiguousarray(done[:, lo:hi]).tobytes()
        assert float(p["tmax"]) == 11.0                       # max over ranks of 10 + rank
        assert tuple(p["total"]) == whole.episode_stats()     # counters add up
    assert whole.episode_stats()[0] > 0
    assert tuple(parts[0]["local"] + parts[1]["local"]) == whole.episode_stats()


def test_shard_and_split_arithmetic():
    assert sharding.shard(0, 8, 65536) == (0, 65536)
    assert sharding.shard(7, 8, 65536) == (7 * 65536, 65536)
    with pytest.raises(ValueError):
        sharding.shard(8, 8, 65536)
    with pytest.raises(ValueError):
        sharding.shard(0, 1 << 20, 1 << 12)
    parts = sharding.split(1000, 3)
    assert parts == [(0, 334), (334, 333), (667, 333)]
    assert sum(n for _, n in sharding.split(65536, 7)) == 65536
    covered = []
    for base, n in sharding.split(65536, 7):
        covered.extend([base, base + n])
    assert covered[0] == 0 and covered[-1] == 65536
    assert all(covered[2 * k + 1] == covered[2 * k + 2] for k in range(6))
    assert sharding.max_over_ranks(3.5) == 3.5 and sharding.sum_stats((1, 2, 3)) == (1, 2, 3)
