"""The N > 1 path of the benchmark on CPU: two gloo ranks shard by sequence (independent
replicas, no data-path exchange), time is the slowest rank's, throughput is the whole job's."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2312_11514_b200 import workloads as W
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = bench.rank_config(W.CONFIGS["tiny"], rank)
    x = W.make_inputs(cfg)                                    # this rank's own sequence
    ms = bench.max_over_ranks(10.0 * (rank + 1), world, "cpu")
    gathered = [None] * world
    dist.all_gather_object(gathered, (cfg.seed, float(x.float().sum())))
    if rank == 0:
        out.put((ms, bench.whole_job_tokens_per_s(50, world, ms), gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_by_sequence_and_report_slowest_rank():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, value, gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ms == 20.0                                          # max over ranks, not the mean
    assert value == 2 * 50 / 0.020                             # both ranks' tokens count
    (seed0, sum0), (seed1, sum1) = gathered
    assert seed0 != seed1 and sum0 != sum1                     # different sequences per rank


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    assert bench.whole_job_tokens_per_s(100, 1, 250.0) == 400.0
