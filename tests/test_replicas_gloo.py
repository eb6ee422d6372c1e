"""The N > 1 path of the benchmark on CPU: two gloo ranks, request sharding and the max-over-ranks
timing reduction."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_03682_b200 import replicas


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        replicas.barrier()
        slowest = replicas.max_over_ranks(10.0 + 5.0 * rank)
        lo, hi = replicas.shard_requests(7, world, rank)
        out.put((rank, slowest, lo, hi))
        replicas.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_replica_and_cover_all_requests():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]
    assert (res[0][2], res[0][3], res[1][2], res[1][3]) == (0, 4, 4, 7)


def test_sharding_is_contiguous_and_balanced():
    for n in (0, 1, 7, 64, 65):
        for world in (1, 2, 3, 8):
            ranges = [replicas.shard_requests(n, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            assert all(ranges[i][1] == ranges[i + 1][0] for i in range(world - 1))
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 1


def test_single_process_helpers_are_no_ops():
    assert replicas.max_over_ranks(3.5) == 3.5
    replicas.barrier()
