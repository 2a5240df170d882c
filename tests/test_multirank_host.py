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


def test_single_process_needs_no_process_group():
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_value(4e9, 1, 2.0) == 4e9 / 2e-3 / 1e9
