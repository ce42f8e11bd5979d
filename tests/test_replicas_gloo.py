"""The multi-GPU mode is independent replicas (no data-path collective). Its rank plumbing -
distinct prompts per replica, max-over-ranks timing, whole-job aggregation - is covered here with
two gloo processes on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    import pop_synth as ps
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env()[:2] == (rank, world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)
    tok = ps.uniform_tokens(bench.replica_seed(rank), 1, 16, 1000)
    gathered = [torch.zeros_like(tok) for _ in range(world)]
    dist.all_gather(gathered, tok)
    out[rank] = (ms, bench.aggregate_tokens_per_s(8192, world, ms), not torch.equal(gathered[0], gathered[1]))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_sum_the_tokens():
    port = 29500 + os.getpid() % 2000
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    for r in range(2):
        ms, value, distinct = out[r]
        assert ms == 15.0
        assert abs(value - 2 * 8192 / 15e-3) < 1e-6
        assert distinct


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_tokens_per_s(100, 1, 50.0) == 2000.0
