"""The multi-rank part of bench.py on CPU: two gloo ranks, max-over-ranks timing and whole-job
throughput of independent replicas (the path has no data-path collective)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    dist.barrier()
    ms = bench.max_over_ranks(local_ms, dist, "cpu")
    value = bench.whole_job_tokens_per_s(world, 1000, ms)
    out.put((rank, ms, value))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_timing_is_max_over_ranks_and_throughput_is_whole_job():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value in results:
        assert ms == 15.0
        assert abs(value - 2 * 1000 / 15e-3) < 1e-6


def test_single_process_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_tokens_per_s(1, 17554, 0.5) == 17554 / 0.5e-3
    c = bench.workload_counts(__import__("workloads").CONFIGS["tiny"], __import__("workloads").prompt_lengths("tiny"))
    # tiny: T = 429, sum l(l+1)/2 = 15 876 visible pairs, 4 heads of 64
    assert c["total_tokens"] == 429 and c["useful_flops"] == 4 * 4 * 64 * 15876
