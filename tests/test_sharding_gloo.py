"""world_size-2 gloo test of the multi-GPU host logic (token sharding, max-over-ranks timing)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2310_04361_b200 import sharding, workloads as wl


def test_token_shards_partition_the_batch():
    for T in (0, 1, 7, 4096, 25216):
        for world in (1, 2, 3, 8):
            spans = [sharding.token_shard(T, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == T
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = wl.with_tokens(wl.CONFIGS["tiny"], 101)
        w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
        b, e = sharding.token_shard(cfg.T, rank, world)
        # each rank runs the layer on its own tokens only (here with the CPU oracle standing in for a GPU)
        part = oracle.layer(x[b:e], w, oracle.ACT_RELU, 0.5)
        np.save(os.path.join(out_dir, f"y{rank}.npy"), part["y"])
        np.save(os.path.join(out_dir, f"k{rank}.npy"), part["k"])
        slow = sharding.max_over_ranks(1.0 + rank)
        thr = sharding.whole_job_throughput(e - b, 1.0 + rank)
        torch.save({"slow": slow, "thr": thr}, os.path.join(out_dir, f"m{rank}.pt"))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_rank_token_sharding_matches_single_rank(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    cfg = wl.with_tokens(wl.CONFIGS["tiny"], 101)
    w, x = wl.make_weights(cfg), wl.make_tokens(cfg)
    full = oracle.layer(x, w, oracle.ACT_RELU, 0.5)
    y = np.concatenate([np.load(tmp_path / f"y{r}.npy") for r in range(world)])
    k = np.concatenate([np.load(tmp_path / f"k{r}.npy") for r in range(world)])
    assert np.array_equal(y, full["y"]) and np.array_equal(k, full["k"])     # tokens are independent
    for r in range(world):
        m = torch.load(tmp_path / f"m{r}.pt")
        assert m["slow"] == 2.0                      # the slowest rank decides
        assert m["thr"] == 101 / 2.0                 # all ranks' units over the slowest time
