"""The N > 1 bookkeeping on CPU: two gloo ranks shard a problem, time it and aggregate the way
bench.py does (max over ranks, whole-job value).  The sharded oracle results must reassemble to
the unsharded result exactly -- the path needs no exchange between ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_11728_b200 import inputs, sharding


def test_shard_ranges_tile_exactly():
    for total in (0, 1, 127, 128, 1000, 100352):
        for world in (1, 2, 3, 8):
            for multiple in (1, 16, 128):
                got = [sharding.shard_range(total, r, world, multiple) for r in range(world)]
                assert got[0][0] == 0 and got[-1][1] == total
                for (a, b), (c, d) in zip(got, got[1:]):
                    assert b == c and a <= b and c <= d
                sizes = [b - a for a, b in got]
                assert max(sizes) - min(sizes) < 2 * multiple
                assert all(a % multiple == 0 or a == total for a, _b in got)
    with pytest.raises(ValueError):
        sharding.shard_range(10, 2, 2)


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
    try:
        from oracle import mip_oracle as orc
        M, N, K = 301, 77, 160
        A = inputs.uniform_s8(M * K, 1)
        B = inputs.uniform_s8(N * K, 2)
        lo, hi = sharding.shard_range(M, rank, world, multiple=16)
        C_part = orc.gemm(A[lo * K:hi * K], B, hi - lo, N, K)          # rows of A and C, all of B
        np.save(os.path.join(out_dir, "part%d.npy" % rank), np.concatenate([[lo, hi], C_part]))
        # timing aggregation as bench.py does it: slowest rank decides, value is the whole job's
        elapsed = 0.5 + 0.25 * rank
        worst = sharding.max_over_ranks(elapsed, dist)
        value = sharding.aggregate_throughput(100.0, elapsed, world, dist)
        assert abs(worst - 0.75) < 1e-12
        assert abs(value - world * 100.0 / 0.75) < 1e-9
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_aggregate(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    from oracle import mip_oracle as orc
    M, N, K = 301, 77, 160
    A = inputs.uniform_s8(M * K, 1)
    B = inputs.uniform_s8(N * K, 2)
    want = orc.gemm(A, B, M, N, K).reshape(M, N)
    got = np.zeros_like(want)
    covered = 0
    for r in range(world):
        part = np.load(os.path.join(str(tmp_path), "part%d.npy" % r))
        lo, hi = int(part[0]), int(part[1])
        got[lo:hi] = part[2:].reshape(hi - lo, N)
        covered += hi - lo
    assert covered == M and np.array_equal(got, want)
    assert sharding.max_over_ranks(3.0) == 3.0          # no process group: identity
