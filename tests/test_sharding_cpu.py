"""Multi-rank host logic on CPU (gloo, world size 2): a batch of groups is split
into contiguous per-rank blocks, every rank processes its block on its own,
and the concatenation of the per-rank results equals the unsharded result.
There is no exchange step on the data path; the only collective here is the
test's own all_gather of the results.  (No GPU in this test: the per-rank
compute is the CPU checker standing in for the rank's GPU.)"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2109_09868_b200.sharding import shard_groups


def test_shard_groups_partitions_exactly():
    for G in (0, 1, 7, 64, 65536, 262144 + 3):
        for world in (1, 2, 3, 8):
            blocks = [shard_groups(G, world, r) for r in range(world)]
            assert blocks[0][0] == 0
            for (s0, n0), (s1, n1) in zip(blocks, blocks[1:]):
                assert s1 == s0 + n0 and n0 >= n1 >= n0 - 1
            assert blocks[-1][0] + blocks[-1][1] == G
    with pytest.raises(ValueError):
        shard_groups(10, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, G, out_path):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2109_09868_b200 import workloads as wl

    oracle.set_threads(1)
    w = wl.workload(2, G)
    Yt = wl.gaussian_predictions(w, "cpu").numpy()  # every rank can regenerate the seeded batch
    mask = wl.masks(w)
    start, count = shard_groups(G, world, rank)
    mine, n_used, _ = oracle.decode(w.K, w.W, Yt[start:start + count], mask[start:start + count])
    # gather the per-rank blocks (padded to the largest block) in rank order
    biggest = shard_groups(G, world, 0)[1]
    pad = torch.zeros((biggest, w.K, w.C), dtype=torch.float64)
    pad[:count] = torch.from_numpy(mine)
    parts = [torch.zeros_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad)
    if rank == 0:
        whole = torch.cat([parts[r][: shard_groups(G, world, r)[1]] for r in range(world)]).numpy()
        ref, _, _ = oracle.decode(w.K, w.W, Yt, mask)
        np.save(out_path, np.array([float(np.abs(whole - ref).max()), whole.shape[0]]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_over_gloo_reproduce_the_unsharded_result(tmp_path):
    out = str(tmp_path / "result.npy")
    G = 101  # odd: the two blocks differ in size
    mp.spawn(_rank_main, args=(2, _free_port(), G, out), nprocs=2, join=True)
    err, n = np.load(out)
    assert n == G and err == 0.0
