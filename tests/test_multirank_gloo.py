"""N > 1 host logic on CPU: gloo, world size 2.  Heads are sharded over ranks without any data-path
collective; each rank evaluates its shard (here with the oracle, standing in for the GPU call), the shards
tile the full result, and the timing reduction takes the MAX over ranks."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_17419_b200 import sharding


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, outdir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import kata_oracle as ko
    from paper_2607_17419_b200 import inputs
    w = inputs.gaussian_workload("mr", "f32", 1, 5, 96, 8, 8, 64, 77)
    lo, hi = sharding.pair_range(w.B * w.H, rank, world)
    q = w.q_ref.reshape(-1, w.T, w.d_k)
    k = w.k_ref.reshape(-1, w.T, w.d_k)
    v = w.v_ref.reshape(-1, w.T, w.d_v)
    mine = np.stack([ko.kata_chunked(q[i], k[i], v[i], 64) for i in range(lo, hi)])
    np.save(os.path.join(outdir, f"shard{rank}.npy"), mine)
    ms = sharding.max_over_ranks([10.0 + 5.0 * rank, 3.0 - rank])
    assert ms == [10.0 + 5.0 * (world - 1), 3.0]
    dist.barrier()
    dist.destroy_process_group()


def test_pair_range_partitions():
    for n in (0, 1, 5, 16, 17, 128):
        for world in (1, 2, 3, 8):
            ranges = [sharding.pair_range(n, r, world) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 1
    assert sharding.whole_job_rate(131072, 4, 8.0) == 4 * 131072 / 8e-3


def test_two_ranks_tile_the_full_result(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    from oracle import kata_oracle as ko
    from paper_2607_17419_b200 import inputs
    w = inputs.gaussian_workload("mr", "f32", 1, 5, 96, 8, 8, 64, 77)
    full = ko.batched(ko.kata_quadratic, w.q_ref, w.k_ref, w.v_ref).reshape(-1, w.T, w.d_v)
    got = np.concatenate([np.load(os.path.join(tmp_path, f"shard{r}.npy")) for r in range(world)])
    assert got.shape == full.shape
    assert np.max(np.abs(got - full)) < 1e-10
