"""The N > 1 path of bench.py on CPU: two gloo ranks exercise the shard assignment, the
max-over-ranks timing reduction and the aggregate-throughput arithmetic (the data path itself
has no collective: every rank solves its own matrices)."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2505_23949_b200 import synth
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        total = bench.max_over_ranks(local_ms, world)
        idx = bench.rank_workload_index(rank)
        a = synth.gaussian_abs(8, 16, 0.02, 1000 * 4 + idx)
        gathered = [None] * world
        dist.all_gather_object(gathered, (idx, float(a.sum()), total))
        if rank == 0:
            out.put(gathered)
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_distinct_shards_and_the_slowest_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[0] for g in gathered] == [0, 1]             # one workload copy per rank
    assert gathered[0][1] != gathered[1][1]               # different seeds -> different data
    assert all(g[2] == 15.0 for g in gathered)            # every rank sees the maximum
    sys.path.insert(0, ROOT)
    import bench
    # 2 ranks x 100 blocks x 3 steps in 15 ms
    assert bench.aggregate_rate(100, 3, 2, 15.0) == 2 * 100 * 3 / 0.015
    assert bench.max_over_ranks(7.0, 1) == 7.0


def test_reference_arm_is_rank0_only(tmp_path):
    sys.path.insert(0, ROOT)
    import bench

    class A:
        steps, warmup, gpus = 1, 0, 2
    assert bench.run_reference(A, rank=1) is None         # other ranks exit without work
