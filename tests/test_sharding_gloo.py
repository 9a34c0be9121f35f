"""The multi-GPU path is a batch partition with no data-path collective; its host logic
(shard ranges, slowest-rank timing, whole-job throughput) is covered here with two gloo
ranks on the CPU."""
import os
import socket

import pytest
import torch.multiprocessing as mp

from paper_1911_02150_b200 import sharding


def test_shard_ranges_partition_the_batch():
    for n in (1, 7, 32, 256, 1000):
        for world in (1, 2, 3, 8):
            ranges = [sharding.shard_range(n, r, world) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n
            for (a0, a1), (b0, b1) in zip(ranges[:-1], ranges[1:]):
                assert a1 == b0
            sizes = [e - s for s, e in ranges]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_range(4, 2, 2)


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sharding.init_process_group("gloo")
    assert sharding.world_from_env() == (rank, rank, world)
    start, end = sharding.shard_range(33, rank, world)
    sharding.barrier()
    seconds = 2.0 if rank == 0 else 3.0                 # rank 1 is the slow one
    thr, slow = sharding.aggregate_throughput(float(end - start), seconds)
    out.put((rank, start, end, thr, slow, sharding.max_over_ranks(float(rank))))
    sharding.barrier()


def test_two_gloo_ranks_agree_on_the_slowest_rank_and_total():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, e0, thr0, slow0, mx0), (r1, s1, e1, thr1, slow1, mx1) = got
    assert (s0, e0, s1, e1) == (0, 17, 17, 33)
    assert slow0 == slow1 == 3.0
    assert thr0 == thr1 == pytest.approx(33 / 3.0)
    assert mx0 == mx1 == 1.0
