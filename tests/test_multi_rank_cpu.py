"""The multi-GPU path has no data-path collective: ranks take (batch, head)
shards and only timings are reduced.  These tests run that plumbing with two
gloo ranks on the CPU."""

import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2401_09486_b200 import multi_gpu


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # each rank owns a disjoint slice of the 1024 (batch, head) pairs and "times" its own work
        own = multi_gpu.shard_range(1024 + 1, rank, world)
        times = [10.0 + rank, 3.0 - rank, float(len(own))]
        red = multi_gpu.max_over_ranks(times)
        gathered = [None] * world
        dist.all_gather_object(gathered, (list(own)[:1] + list(own)[-1:], len(own), multi_gpu.rank_seed(1000, rank, 2)))
        out.put((rank, red, gathered))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_pairs_and_take_max_times():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, red, gathered in results:
        assert red == [11.0, 3.0, 513.0]                       # element-wise max over the two ranks
        (e0, n0, s0), (e1, n1, s1) = gathered
        assert n0 + n1 == 1025 and e0 == [0, 512] and e1 == [513, 1024]   # disjoint, contiguous, complete
        assert s0 != s1
    assert multi_gpu.job_throughput(100.0, 2, 50.0) == pytest.approx(4000.0)


@pytest.mark.parametrize("n,world", [(1024, 8), (10, 3), (2, 4), (0, 2)])
def test_shard_range_partitions_exactly(n, world):
    seen = []
    for r in range(world):
        seen += list(multi_gpu.shard_range(n, r, world))
    assert seen == list(range(n))
    sizes = [len(multi_gpu.shard_range(n, r, world)) for r in range(world)]
    assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        multi_gpu.shard_range(n, world, world)


def test_max_over_ranks_without_process_group_is_identity():
    assert multi_gpu.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
