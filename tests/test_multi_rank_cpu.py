"""N > 1 host logic on CPU: two gloo ranks shard the sequences, time their own (simulated) step
loops, and agree on the max-over-ranks time and the whole-job throughput."""
import os
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    from paper_2511_11907_b200 import shard
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        seqs = list(shard.sequences_of_rank(4, rank))
        elapsed_ms = 10.0 + 5.0 * rank                   # rank 1 is the slower one
        dist.barrier()
        worst, = shard.max_over_ranks([elapsed_ms])
        value = shard.aggregate_throughput(1.0, 20, worst, world)
        q.put((rank, seqs, shard.rank_seed_offset(rank), worst, value))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_time_and_throughput():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, o0, w0, v0), (r1, s1, o1, w1, v1) = results
    assert s0 == [0, 1, 2, 3] and s1 == [4, 5, 6, 7] and o0 != o1      # disjoint shards, distinct seeds
    assert w0 == w1 == 15.0                                            # both see the slowest rank's time
    assert v0 == v1 == 2 * 20 / 0.015


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2511_11907_b200 import shard
    assert shard.max_over_ranks([3.0, 4.5]) == [3.0, 4.5]
    assert shard.aggregate_throughput(2.0, 10, 100.0, 1) == 200.0
