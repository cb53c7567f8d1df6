"""The N > 1 path on CPU: two gloo ranks take disjoint head slices of one
attention call (oracle arithmetic stands in for the kernel here) and their
concatenation equals the single-rank result; no data-path collective is needed."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_26538_b200.sharding import unit_slice


def test_unit_slice_partitions():
    for n in (0, 1, 7, 24, 25):
        for world in (1, 2, 3, 8):
            cuts = [unit_slice(n, world, r) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
            sizes = [b - a for a, b in cuts]
            assert max(sizes) - min(sizes) <= 1


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import hilberta_oracle as orc
    H, tile, o, hs, nt, heads, D = 8, 16, 4, 2, 5, 6, 16
    S = nt + H * H
    g = torch.Generator().manual_seed(9)
    q, k, v = (torch.randn((1, heads, S, D), generator=g).numpy() for _ in range(3))
    M = orc.mask(H, H, tile, o, hs, nt)
    lo, hi = unit_slice(heads, world, rank)
    part = orc.attention(q[:, lo:hi], k[:, lo:hi], v[:, lo:hi], M)
    np.save(os.path.join(out_dir, f"part{rank}.npy"), part)
    # the only cross-rank traffic is the timing reduction the bench does
    t = torch.tensor([float(rank + 1)])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert t.item() == world
    dist.barrier()
    if rank == 0:
        full = orc.attention(q, k, v, M)
        parts = [np.load(os.path.join(out_dir, f"part{r}.npy")) for r in range(world)]
        assert np.array_equal(np.concatenate(parts, axis=1), full)
    dist.destroy_process_group()


def test_two_ranks_head_sharding(tmp_path):
    mp.spawn(_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
