"""The N > 1 path of the benchmark on CPU: two gloo ranks shard by sequence (independent
replicas, no data-path exchange), time is the slowest rank's, throughput is the whole job's."""
import json
import os
import socket
import subprocess
import sys

import pytest

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


# ---------------------------------------------------------------- neuron sharding (two ranks)
def _shard_worker(rank, world, port, out):
    """Each rank takes its share of one layer with the product's own host logic
    (runtime.neuron_shard, workloads.slice_layer), computes the share's partial outputs (the
    oracle stands in for the CUDA step, which needs a GPU) and sums them over gloo with
    runtime.sum_partial_outputs.  Rank 0 reports the sums and its share's bounds."""
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import lif_oracle as O
    from paper_2312_11514_b200 import runtime as R
    from paper_2312_11514_b200 import workloads as W
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = W.CONFIGS["tiny"]
    w = W.make_layer(cfg, 0)
    lo, hi = R.neuron_shard(cfg.d_ff, rank, world)
    mine = W.slice_layer(w, lo, hi)
    assert mine["bundles"].shape == (hi - lo, 2 * cfg.d_model) and mine["bundles"].is_contiguous()
    assert mine["B"].shape == (cfg.rank, hi - lo) and mine["B"].is_contiguous()
    assert mine["A"] is w["A"]
    b_down = (torch.arange(cfg.d_model, dtype=torch.float32) / 64).to(torch.float16).numpy()
    cache = O.NeuronCache(cfg.d_model, hi - lo, hi - lo, cfg.window_k)
    X = W.make_inputs(cfg)
    sums, loaded = [], 0
    for t in range(8):
        x = X[t].numpy()
        _, _, lists, y = O.decode_step(cache, x, mine["A"].numpy(), mine["B"].numpy(),
                                       mine["c"].numpy(), 0.0, mine["bundles"].numpy(),
                                       mine["bias_up"].numpy(), b_down if rank == 0 else None)
        loaded += len(lists["load_ids"])
        sums.append(R.sum_partial_outputs(torch.from_numpy(y)).numpy().copy())
    counts = [None] * world
    dist.all_gather_object(counts, (lo, hi, loaded))
    if rank == 0:
        out.put((np.stack(sums), counts))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_by_neuron_and_sum_their_partial_outputs():
    import numpy as np
    from oracle import lif_oracle as O
    from paper_2312_11514_b200 import workloads as W
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_shard_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    sums, counts = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = W.CONFIGS["tiny"]
    assert [(lo, hi) for lo, hi, _ in counts] == [(0, cfg.d_ff // 2), (cfg.d_ff // 2, cfg.d_ff)]
    # one device holding every neuron
    w = W.make_layer(cfg, 0)
    b_down = (torch.arange(cfg.d_model, dtype=torch.float32) / 64).to(torch.float16).numpy()
    cache = O.NeuronCache(cfg.d_model, cfg.d_ff, cfg.d_ff, cfg.window_k)
    X = W.make_inputs(cfg)
    loaded = 0
    for t in range(8):
        _, _, lists, y = O.decode_step(cache, X[t].numpy(), w["A"].numpy(), w["B"].numpy(),
                                       w["c"].numpy(), 0.0, w["bundles"].numpy(),
                                       w["bias_up"].numpy(), b_down)
        loaded += len(lists["load_ids"])
        np.testing.assert_allclose(sums[t], y, rtol=1e-11, atol=1e-12)
    assert sum(n for _, _, n in counts) == loaded           # host-link traffic splits, never doubles


def test_neuron_shares_are_equal_multiples_of_eight():
    import pytest
    from paper_2312_11514_b200 import runtime as R
    with pytest.raises(ValueError):
        R.neuron_shard(1000, 0, 3)
    with pytest.raises(ValueError):
        R.neuron_shard(1024, 2, 2)
    assert R.neuron_shard(1024, 3, 4) == (768, 1024)
    assert R.sum_partial_outputs(torch.ones(2, 4)).tolist() == [[1.0] * 4] * 2   # one device: no-op


def test_bench_starts_its_own_ranks_for_gpus_above_one():
    # `bench.py --gpus 2` outside torchrun starts two ranks itself (here: the device-free stub arm
    # over gloo); rank 0 prints one line for the whole job, with the slowest rank's time
    bench = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "bench.py")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, bench, "--gpus", "2", "--impl", "stub", "--steps", "6", "--warmup", "3"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2 and rec["steps"] == 6 and rec["scaling"] == "weak"
    # rank 1 sleeps 2 ms per token: the job's time is the slowest rank's, the rate counts both ranks
    assert rec["ms_per_step"] >= 2.0
    assert rec["value"] == pytest.approx(2 * 6 / (rec["ms_per_step"] * 6 / 1e3), rel=1e-9)
    # one rank: no launcher involved, same line shape
    res1 = subprocess.run([sys.executable, bench, "--gpus", "1", "--impl", "stub", "--steps", "4", "--warmup", "3"],
                          capture_output=True, text=True, timeout=120, env=env)
    assert res1.returncode == 0 and json.loads(res1.stdout.splitlines()[-1])["n_gpus"] == 1


def test_bench_refuses_more_gpus_than_the_node_has():
    import torch
    have = torch.cuda.device_count() if torch.cuda.is_available() else 0
    bench = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "bench.py")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, bench, "--gpus", str(have + 2), "--steps", "3"],
                         capture_output=True, text=True, timeout=120, env=env)
    assert res.returncode == 2 and "CUDA devices" in res.stderr and not res.stdout.strip()
