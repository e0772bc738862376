"""The multi-process plumbing (barrier, max-over-ranks timing, unit sharding) on two gloo ranks."""
import os
import socket

import pytest
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2609_09208_b200 import dist_util
    r, w = dist_util.init_from_env("gloo")
    assert (r, w) == (rank, world)
    dist_util.barrier()
    # rank 1 is "slower": the job's time is the maximum, its work the sum
    thr, worst = dist_util.aggregate_throughput(units_this_rank=1000.0 * (rank + 1), elapsed_ms_this_rank=10.0 * (rank + 1))
    shard = dist_util.shard_units(7, rank, world)
    out.put((rank, thr, worst, list(shard)))
    dist_util.barrier()
    import torch.distributed as dist
    dist.destroy_process_group()


def test_two_rank_aggregation_and_sharding():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, thr, worst, shard in res:
        assert worst == 20.0                       # max over ranks
        assert thr == pytest.approx(3000.0 / 0.020)  # all units / slowest rank's time
    assert res[0][3] + res[1][3] == list(range(7))  # disjoint, complete, ordered shards


def test_single_process_is_a_no_op():
    from paper_2609_09208_b200 import dist_util
    assert dist_util.max_over_ranks(3.5) == 3.5
    assert dist_util.aggregate_throughput(10.0, 5.0) == (2000.0, 5.0)
    assert list(dist_util.shard_units(5, 0, 1)) == [0, 1, 2, 3, 4]
