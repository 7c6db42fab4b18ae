"""The N > 1 path of the benchmark on CPU: two gloo ranks shard the rows of a
product, each checks its shard against the oracle computed for exactly those
rows, and the timing reduction takes the slowest rank."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2506_09092_b200 import sharding  # noqa: E402


def test_row_shards_partition_the_rows():
    for M in (0, 1, 7, 4096, 4097, 3001):
        for world in (1, 2, 3, 8):
            cuts = [sharding.row_shard(M, r, world) for r in range(world)]
            assert cuts[0][0] == 0 and cuts[-1][1] == M
            assert all(cuts[i][1] == cuts[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in cuts]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.row_shard(10, 2, 2)
    assert sharding.weak_scaling_rows(4096, 8) == 32768
    assert sharding.aggregate_throughput(10.0, 4, 2.0) == 20.0
    assert sharding.max_over_ranks(3.5) == 3.5          # no process group: identity


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import oracle
    from paper_2506_09092_b200 import inputs as gi
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        M, N, K = 37, 19, 23
        rng = np.random.default_rng(5)                       # same operands on every rank
        A = gi.f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))
        Bm = gi.f32_to_bf16_bits(rng.standard_normal((K, N)).astype(np.float32))
        b, e = sharding.row_shard(M, rank, world)
        C_shard, _ = oracle.gemm(np.ascontiguousarray(A[b:e]), Bm, e - b, N, K)
        # gather the shards and compare with the unsharded product
        full = torch.zeros(M, N, dtype=torch.float64)
        full[b:e] = torch.from_numpy(C_shard)
        dist.all_reduce(full)                                # shards are disjoint: sum = concatenation
        C_all, _ = oracle.gemm(A, Bm, M, N, K)
        same = bool(np.array_equal(full.numpy(), C_all))
        slowest = sharding.max_over_ranks(1.0 + rank)        # rank r "took" 1 + r seconds
        dist.barrier()
        out.put((rank, same, slowest, (b, e)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_rows_and_reduce_timing():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    results.sort()
    assert [r[1] for r in results] == [True, True]
    assert [r[2] for r in results] == [2.0, 2.0]             # both see the slowest rank's time
    assert results[0][3] == (0, 19) and results[1][3] == (19, 37)
