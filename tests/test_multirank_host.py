"""Host-side logic of the N > 1 benchmark path, on CPU with two gloo ranks.

The path does not shard (every rank runs an independent replica), so the only multi-rank code is the
rendezvous, the barrier and the max-over-ranks reduction of the step time.
"""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank), LC_BENCH_BACKEND="gloo")
    r, w, lr = bench.dist_setup(world)
    assert (r, w, lr) == (rank, world, rank)
    bench.barrier()
    local_ms = 10.0 + 5.0 * rank  # rank 1 is the slow replica
    worst = bench.max_over_ranks(local_ms)
    value = bench.aggregate_value(8e9, w, worst)
    results[rank] = (worst, value)
    bench.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_replica():
    world = 2
    port = _free_port()
    mgr = mp.Manager()
    results = mgr.dict()
    mp.spawn(_worker, args=(world, port, results), nprocs=world, join=True)
    assert results[0] == results[1]
    worst, value = results[0]
    assert worst == 15.0
    assert abs(value - 2 * 8e9 / 15e-3 / 1e9) < 1e-6


def _stats_buffer(oracle, base, cur):
    """The 8 KB statistics buffer of lc_shard_stats, rebuilt on the CPU from the oracle's bins: 512 counts (u64), then per
    key the running maxima of ~bits and of bits over the bucket (0 for an empty bucket)."""
    import numpy as np

    count, mmin, mmax = oracle.bins(base, cur)
    key = np.arange(512, dtype=np.uint64)
    lo_bits = ((key << np.uint64(23)) | mmin.astype(np.uint64)).astype(np.uint32)
    hi_bits = ((key << np.uint64(23)) | mmax.astype(np.uint64)).astype(np.uint32)
    inv_min = np.where(count > 0, ~lo_bits, np.uint32(0)).astype(np.uint32)
    max_bits = np.where(count > 0, hi_bits, np.uint32(0)).astype(np.uint32)
    return np.concatenate([count.view(np.uint8), inv_min.view(np.uint8), max_bits.view(np.uint8)])


def _shard_worker(rank, world, port, results):
    import numpy as np

    from oracle import lc_oracle
    from paper_2009_13003_b200 import binding

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group(backend="gloo")
    rng = np.random.default_rng(5)  # the same vector on every rank; each takes its shard
    n = 30_000
    base = rng.normal(0, 0.02, n).astype(np.float32)
    cur = (base + rng.laplace(0, 1e-3, n).astype(np.float32) * np.where(np.arange(n) < n // 2, 50.0, -1.0).astype(np.float32))
    lo, hi = (0, n // 2) if rank == 0 else (n // 2, n)
    mine = torch.from_numpy(_stats_buffer(lc_oracle, base[lo:hi], cur[lo:hi]).copy())
    got = binding.all_reduce_stats(mine).numpy()
    results[rank] = bool(np.array_equal(got, _stats_buffer(lc_oracle, base, cur)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_exchange_the_bucket_statistics_of_their_shards():
    # the one exchange step of a vector split over devices: after it every rank holds the whole vector's statistics
    world = 2
    mgr = mp.Manager()
    results = mgr.dict()
    mp.spawn(_shard_worker, args=(world, _free_port(), results), nprocs=world, join=True)
    assert results[0] is True and results[1] is True


def test_single_process_needs_no_process_group():
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_value(4e9, 1, 2.0) == 4e9 / 2e-3 / 1e9
