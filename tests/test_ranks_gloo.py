"""The N > 1 host logic on CPU: two gloo ranks shard a batch, draw their own seeded workloads, and
combine per-rank timings the way bench.py does (units of all ranks / slowest rank's time)."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2312_04985_b200 import ranks, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert ranks.env_rank() == (world, rank, rank)
        begin, end = ranks.shard_batch(5, world, rank)
        case = synth.make_case("c2", B=end - begin, Hq=2, Hkv=2, S=64, seed=ranks.rank_seed(2, rank))
        seconds = 0.5 + rank          # rank 1 is the slow one
        tput = ranks.whole_job_throughput(case.B * case.Hq, seconds)
        out.put((rank, begin, end, float(case.K.float().sum()), ranks.max_over_ranks(seconds), tput))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_and_aggregate():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, b0, e0, s0, m0, t0), (r1, b1, e1, s1, m1, t1) = res
    assert (b0, e0, b1, e1) == (0, 3, 3, 5)                  # 5 sequences over 2 ranks: 3 + 2, no overlap, no gap
    assert s0 != s1                                           # each rank drew its own batch
    assert m0 == m1 == 1.5                                    # slowest rank's time, seen by both
    assert t0 == t1 == (3 * 2 + 2 * 2) / 1.5                  # all ranks' units / slowest time


def test_single_process_helpers():
    assert ranks.shard_batch(64, 8, 3) == (24, 32)
    assert [ranks.shard_batch(10, 4, r) for r in range(4)] == [(0, 3), (3, 6), (6, 8), (8, 10)]
    assert ranks.max_over_ranks(2.5) == 2.5 and ranks.whole_job_throughput(10, 2.0) == 5.0
