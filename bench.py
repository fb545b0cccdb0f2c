"""Benchmark of the sparse-decode FFN stack (predict -> window update -> bundle fetch ->
sparse FFN, every layer, one token per step) on seeded synthetic data.

  python bench.py --gpus N --steps K --warmup W           CUDA path, one JSON line
  python bench.py --impl reference ...                     CPU oracle on the host cores
  python bench.py --floors                                 link and launch reference points

One step = one decode token through all layers of the configuration.  `value` is tokens/s
with the decode inputs resident in HBM (the bundle store stays in pinned host memory: reading
it is part of the method); `e2e` passes pinned HOST inputs/outputs through
lif_graph_launch_host.  A token is one CUDA graph (lif_graph_capture).  Per-kernel durations
for the roofline come from a further pass after the timed tokens: for each kernel, a graph of
that one kernel on every layer (the lists of the last token) is replayed and timed with CUDA
events.  With --gpus N > 1 and no torchrun environment the script starts its own N ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "ffn_stack_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum over algorithmic bytes of sparse_ffn_kernel, from
# the ncu capture summarised under profiles/ (set to None when that kernel changes)
FFN_TRAFFIC_RATIO = 1.003
# fetch_ffn_kernel: bytes read from system memory per bundle byte, same kind of capture
FETCH_TRAFFIC_RATIO = 1.000
FALLBACK_HBM_GBS = 6650.0
_LINK_PEAK = {}          # measured pinned host -> device rate per local device, GB/s


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(index), "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL,
                text=True)
        except OSError:
            pass

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        out, _ = self.proc.communicate(timeout=10)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


def rank_config(cfg, rank):
    """Each rank decodes its own sequence with its own replica of the stack: independent
    problems, so sharding is by sequence and needs no exchange on the data path."""
    return cfg.scaled(seed=cfg.seed + 100 * rank) if rank else cfg


def max_over_ranks(ms, world, device):
    """Slowest rank's time (MAX all-reduce over the default process group)."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(steps, world, ms_slowest):
    """Weak scaling: every rank processed `steps` tokens in at most ms_slowest."""
    return world * steps / (ms_slowest / 1e3)


GATE_MODES = {"none": 0, "bundled": 1, "resident": 2}


def workload_string(cfg, n_layers, gate_name, gate_mode, act_thr):
    return (f"{cfg.name}: {n_layers} layers d_model={cfg.d_model} d_ff={cfg.d_ff} rank={cfg.rank} "
            f"window_k={cfg.window_k} streams={cfg.n_streams}, AR(1) decode inputs"
            + (f", gated FFN ({gate_name} gate, FATReLU {act_thr})" if gate_mode else ""))


def _gate_setup(args):
    """(gate_mode, activation, threshold): gated runs use FATReLU on the gate value (Appendix C,
    Llama 2); ungated runs use ReLU."""
    gm = GATE_MODES[args.gate]
    return (gm, 2, args.act_threshold) if gm else (0, 0, 0.0)


def _inputs(cfg, n_tokens, device, W):
    return W.make_inputs(cfg.scaled(steps=max(cfg.steps, n_tokens)), device=device)[:n_tokens]


# ------------------------------------------------------------------------------ CUDA arm
def run_ours(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    out = measure(args, args.config, args.steps, args.warmup, rank, world, local, detail=True)
    if rank == 0:
        if args.other_configs and world == 1 and args.config == "opt6p7b" and not args.layers \
                and args.gate == "none" and args.shard == "sequences":
            # the other single-GPU configurations at reduced length, so that their numbers are
            # in the same record (batched8 keeps 36.75 GiB of bundles in pinned host memory)
            out["other_configs"] = []
            for name in ("falcon7b", "phi2", "batched8"):
                o = measure(args, name, 24, 8, rank, world, local, detail=False)
                out["other_configs"].append({k: o[k] for k in (
                    "value", "unit", "ms_per_step", "steps", "warmup", "config", "e2e", "roofline",
                    "host_link", "per_token", "kernel_us_per_launch")})
        print(json.dumps(out), flush=True)
    if dist.is_initialized():
        dist.destroy_process_group()


def measure(args, config_name, steps, warmup, rank, world, local, detail):
    """Build the stack of one configuration, time it, and return the record (rank 0)."""
    import torch
    import torch.distributed as dist
    from paper_2312_11514_b200 import binding as B
    from paper_2312_11514_b200 import runtime as R
    from paper_2312_11514_b200 import workloads as W

    dev = f"cuda:{local}"

    # every rank decodes its own sequence with its own replica of the stack (weak scaling,
    # no exchange between ranks)
    # --shard neurons (N > 1): all ranks decode ONE sequence, each with its share of every
    # layer's neurons, and sum their partial outputs after every layer (strong scaling)
    # (at N = 1 the same layer-by-layer path runs with the whole layer as the only share)
    sharded = args.shard == "neurons"
    cfg = W.CONFIGS[config_name]
    cfg = cfg if sharded else rank_config(cfg, rank)
    K, Wm = steps, warmup
    n_tok = Wm + K
    gate_mode, activation, act_thr = _gate_setup(args)
    layers = R.build_stack(cfg, dev, n_layers=args.layers, gate_mode=gate_mode, activation=activation,
                           activation_threshold=act_thr, append_first=args.append_first,
                           shard=(rank, world) if sharded else None)
    handles = [l.handle for l in layers]
    for item in args.tune:                 # launch-shape knobs of include/lif_profile.h
        key, value = item.split("=")
        for h in handles:
            B.lif_set_tuning(h, getattr(B, "TUNE_" + key.upper()), int(value))
    L, S, d = len(layers), cfg.n_streams, cfg.d_model
    X = _inputs(cfg, n_tok, dev, W)
    Y = torch.empty(L, S, d, dtype=torch.float32, device=dev)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def reset():
        for h in handles:
            B.lif_reset(h, sc)

    def stats_sum():
        st = [B.lif_get_stats(h) for h in handles]
        assert all(s.status == B.LIF_OK for s in st), "device status not OK"
        return (sum(s.bytes_fetched for s in st), sum(s.rows_active for s in st),
                sum(s.rows_moved for s in st), sum(s.rows_cached for s in st))

    def slowest(ms):
        return max_over_ranks(ms, world, dev)

    # One CUDA graph holds a whole token (every layer's kernels, both streams); the token's
    # input is copied into dev_x before each launch.
    dev_x = torch.empty(S, d, dtype=torch.float16, device=dev)
    graph = B.lif_graph_capture(handles, dev_x, Y, sc, sf)

    exchange = None
    if sharded and args.exchange == "peer":
        if world == 1 and not dist.is_initialized():      # the buffer mapping needs a group
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            os.environ.setdefault("MASTER_PORT", "29517")
            dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device(dev))
        exchange = R.PeerExchange(L, S, d, dev)

    def layers_then_sums():
        # neuron-sharded token: a layer's output exists only after the exchange, so the layers
        # are launched one by one with the sum over ranks between them (no whole-token graph)
        for l in range(L):
            if exchange is None:                          # library all-reduce, in place
                B.lif_decode_step(handles[l], dev_x, Y[l], sc, sf)
                R.sum_partial_outputs(Y[l])
            else:                                         # peers' partials read by our kernel
                B.lif_decode_step(handles[l], dev_x, exchange.partials[l], sc, sf)
                exchange.sum_layer(l, Y[l], sc)
        if exchange is not None:
            exchange.end_token()

    def token(t):
        with torch.cuda.stream(sc):
            dev_x.copy_(X[t], non_blocking=True)
            if sharded:
                layers_then_sums()
        if not sharded:
            B.lif_graph_launch(graph, sc)

    def token_host(t):
        if not sharded:
            B.lif_graph_launch_host(graph, host_x[t], host_y, sc)
            return
        with torch.cuda.stream(sc):
            dev_x.copy_(host_x[t], non_blocking=True)
            layers_then_sums()
            host_y.copy_(Y, non_blocking=True)
        sc.synchronize()

    # ---- pass 1: device-resident inputs ------------------------------------------------------
    reset()
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record(sc)
    token(0)                 # cold cache: the first token brings in its whole active set
    c1.record(sc)
    for t in range(1, Wm):
        token(t)
    barrier()
    ms_cold = c0.elapsed_time(c1)
    cold_fetched = sum(B.lif_get_stats(h).bytes_fetched for h in handles)
    s0 = stats_sum()
    clocks = ClockSampler(local) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(sc)
    for t in range(Wm, n_tok):
        token(t)
    e1.record(sc)
    barrier()
    ms_total = slowest(e0.elapsed_time(e1))
    clock_info = clocks.stop() if clocks else None
    s1 = stats_sum()
    fetched, rows_active, rows_moved = (s1[i] - s0[i] for i in range(3))

    # ---- pass 2: pinned host inputs and outputs through lif_graph_launch_host ----------------
    host_x = torch.empty(n_tok, S, d, dtype=torch.float16, pin_memory=True)
    host_x.copy_(X)
    host_y = torch.empty(L, S, d, dtype=torch.float32, pin_memory=True)
    reset()
    for t in range(Wm):
        token_host(t)
    barrier()
    e0.record(sc)
    for t in range(Wm, n_tok):
        token_host(t)
    e1.record(sc)
    barrier()
    ms_e2e = slowest(e0.elapsed_time(e1))

    # ---- pass 3: per-kernel durations.  The window state now holds the last token; for each
    # kernel, a graph of that one kernel on every layer (its real lists, the launch shape of the
    # decode step, L2-cold because the layers' rows differ) is replayed and timed with events.
    last = n_tok - 1
    with torch.cuda.stream(sc):
        dev_x.copy_(X[last])
    cnts = torch.stack([l.counts[:16] for l in layers]).cpu()
    n_act_l, n_load_l, n_hit_l, n_used_l = (cnts[:, i].sum().item() for i in (
        B.CNT_N_ACTIVE, B.CNT_N_LOAD, B.CNT_N_HITS, B.CNT_NUM_USED))
    kernel_us = {}
    reps = 20
    if S == 1:
        launchers = {name: (lambda l, kind=kind: B.lif_profile_launch(handles[l], kind, dev_x, Y[l], sc))
                     for kind, name in enumerate(B.KERNELS)
                     if not (gate_mode == B.GATE_RESIDENT and name == "predict_z")}
        if not detail:
            launchers = {k: v for k, v in launchers.items() if k in ("fetch", "ffn_active", "ffn_hits", "ffn_new")}
        if args.append_first == 0 and "ffn_cache" in launchers:
            pass      # rows [0, num_used) are the cache in both orders once a step is complete
    else:
        # several streams: the staged entry points (predictor = 2 kernels; FFN = the tensor-core
        # up, down and partial-sum kernels over all active rows)
        acts = torch.empty(cfg.d_ff, dtype=torch.int32, device=dev)
        nact = torch.zeros(1, dtype=torch.int32, device=dev)
        slot_views = [l._view("active_slots", cfg.d_ff) for l in layers]
        launchers = {
            "predict": lambda l: B.lif_predict(handles[l], dev_x, None, acts, nact, sc),
            "fetch": lambda l: B.lif_fetch_bundles(handles[l], sc),
            "ffn_active": lambda l: B.lif_sparse_ffn(handles[l], dev_x, slot_views[l],
                                                     layers[l].counts[B.CNT_N_ACTIVE:], Y[l], sc),
        }
    for name, launch in launchers.items():
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=sc):
            for l in range(L):
                launch(l)
        with torch.cuda.stream(sc):
            for _ in range(3):
                g.replay()
            e0.record(sc)
            for _ in range(reps):
                g.replay()
            e1.record(sc)
        barrier()
        kernel_us[name] = slowest(e0.elapsed_time(e1)) * 1e3 / (reps * L)
        del g
    n_launch = K * L

    # host-link peak: pinned host -> device cudaMemcpyAsync of 1 GiB, best of 5
    link_peak = _LINK_PEAK.get(local)
    if rank == 0 and link_peak is None:
        nb = 1 << 30
        hbuf = torch.empty(nb, dtype=torch.uint8, pin_memory=True)
        dbuf = torch.empty(nb, dtype=torch.uint8, device=dev)
        best = float("inf")
        for _ in range(5):
            e0.record(); dbuf.copy_(hbuf, non_blocking=True); e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        link_peak = nb / best / 1e6
        _LINK_PEAK[local] = link_peak
        del hbuf, dbuf

    if rank == 0:
        beta = (3 if gate_mode == B.GATE_BUNDLED else 2) * d * 2
        row_extra = 8 if gate_mode == B.GATE_RESIDENT else 2    # bias, or neuron id + gate value
        peak, peak_kind = _peaks()
        # algorithmic bytes of one launch: bundle + bias per row, x in, partials out
        all_bytes = (n_act_l * (beta + row_extra) + L * S * 6 * d) / L
        all_gbs = all_bytes / (kernel_us["ffn_active"] * 1e-6) / 1e9
        if S == 1:
            # the launch the decode step makes: the rows that were already cached (the new rows'
            # terms are added by the fetch kernel, or by a second launch for three-vector bundles)
            ffn_bytes = (n_hit_l * (beta + row_extra) + L * 6 * d) / L
            ffn_us = kernel_us["ffn_hits"]
        else:
            ffn_bytes, ffn_us = all_bytes, kernel_us["ffn_active"]
        ffn_gbs = ffn_bytes / (ffn_us * 1e-6) / 1e9
        fetch_bytes = n_load_l * beta / L
        fetch_gbs = fetch_bytes / (kernel_us["fetch"] * 1e-6) / 1e9
        predictor = None
        if detail or S > 1:
            if gate_mode == B.GATE_RESIDENT:       # gate matrix + bias in, gate values out
                pred_bytes = 2 * cfg.d_ff * d + 2 * cfg.d_ff + 4 * S * cfg.d_ff
                pred_us = kernel_us["predict"] if S > 1 else kernel_us["predict_scores"]
            else:
                pred_bytes = 2 * cfg.rank * (d + cfg.d_ff) + 4 * cfg.d_ff
                pred_us = kernel_us["predict"] if S > 1 else kernel_us["predict_z"] + kernel_us["predict_scores"]
            pred_gbs = pred_bytes / (pred_us * 1e-6) / 1e9
            predictor = {"bound": "hbm", "achieved": pred_gbs, "unit": "GB/s", "frac": pred_gbs / peak,
                         "bytes_per_launch": pred_bytes, "us_per_launch": pred_us}
        split = None
        if S == 1:
            split = {"all_active_rows": {"GBs": all_gbs, "us_per_launch": kernel_us["ffn_active"],
                                         "bytes_per_launch": all_bytes, "frac": all_gbs / peak},
                     "new_rows_GBs": (n_load_l * (beta + row_extra) / L + 6 * d) / (kernel_us["ffn_new"] * 1e-6) / 1e9}
            if "ffn_cache" in kernel_us:
                # the same kernel over every cached row (Section 3.3 item 3 as written)
                cache_bytes = (n_used_l * (beta + row_extra) + L * 6 * d) / L
                cache_gbs = cache_bytes / (kernel_us["ffn_cache"] * 1e-6) / 1e9
                split["whole_cache"] = {"GBs": cache_gbs, "us_per_launch": kernel_us["ffn_cache"],
                                        "bytes_per_launch": cache_bytes, "frac": cache_gbs / peak,
                                        "rows_per_launch": n_used_l / L}
        out = {
            "metric": METRIC, "value": whole_job_tokens_per_s(K, 1 if sharded else world, ms_total), "unit": UNIT,
            "n_gpus": world, "steps": K, "warmup": Wm, "ms_per_step": ms_total / K,
            "higher_is_better": True, "scaling": "strong" if sharded else "weak", "vs_baseline": None,
            "dtype": "f16", "data": "synthetic",
            "config": {"workload": workload_string(cfg, L, args.gate, gate_mode, act_thr),
                       "cache_order": "new neurons stacked first, then the deletions (bundles written "
                                      "straight into freed rows)" if args.append_first else
                                      "deletions first, then new neurons stacked (Section 3.3 as written)",
                       "l2": "per-token working set (all layers' window caches, "
                             f"{s1[3] / n_tok * beta / 2**20:.0f} MiB) exceeds the 126 MB L2",
                       "bundle_store": "pinned host memory, read by the fetch kernel",
                       "parallelism": f"one sequence, neurons of every layer split over {world} GPUs, "
                                      f"partial outputs summed after every layer ({args.exchange})"
                                      if sharded else "independent sequence per GPU"},
            "e2e": {"value": whole_job_tokens_per_s(K, 1 if sharded else world, ms_e2e), "unit": UNIT,
                    "h2d_bytes_per_step": S * d * 2, "d2h_bytes_per_step": L * S * d * 4,
                    "host_link_bytes_per_step": fetched / K},
            # per layer-step: z, scores (or the gate kernel alone), window, moves, fetch (one stream:
            # with the new rows' FFN terms), FFN of cached rows (several streams: up + down), sum
            "gpu_launches": ((7 if S == 1 else 8) - (1 if gate_mode == B.GATE_RESIDENT else 0)
                             + (1 if gate_mode == B.GATE_BUNDLED else 0)) * n_launch,
            "roofline": {"kernel": "sparse_ffn_kernel" if S == 1 else
                                   "ffn_batched_up_kernel + ffn_batched_down_kernel + ffn_reduce_kernel",
                         "bound": "hbm",
                         "achieved": ffn_gbs, "peak": peak, "unit": "GB/s", "frac": ffn_gbs / peak,
                         "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": ffn_gbs / NOMINAL_HBM_GBS,
                         "traffic": FFN_TRAFFIC_RATIO * ffn_bytes
                                    if FFN_TRAFFIC_RATIO and S == 1 and not gate_mode else None,
                         "traffic_how": "dram read+write bytes per algorithmic byte from the ncu capture in "
                                        "profiles/sparse_ffn_kernel_opt6p7b_12layers.md (12 layers, "
                                        "277-463 rows per launch), scaled by this run's rows per launch",
                         "us_per_launch": ffn_us,
                         "bytes_per_launch": ffn_bytes,
                         "how": ("graph of this kernel on every layer, over the rows of the last token "
                                 "that were already cached (the decode step's launch)" if S == 1 else
                                 "graph of these kernels on every layer, over the active rows of the "
                                 "last token") + f", {reps} replays, CUDA events",
                         "other_launches": split},
            "host_link": {"kernel": "fetch_ffn_kernel" if S == 1 and gate_mode != B.GATE_BUNDLED
                                    else "fetch_kernel", "bound": "host_link", "achieved": fetch_gbs,
                          "peak": link_peak, "unit": "GB/s", "frac": fetch_gbs / link_peak,
                          "peak_kind": "of measured (1 GiB pinned cudaMemcpyAsync, this run)",
                          "bytes_per_launch": fetch_bytes, "us_per_launch": kernel_us["fetch"],
                          "traffic": FETCH_TRAFFIC_RATIO * fetch_bytes if S == 1 and not gate_mode else None,
                          "traffic_how": "system-memory bytes read per algorithmic byte from the ncu capture "
                                         "in profiles/fetch_ffn_kernel_opt6p7b_12layers.md, scaled by this "
                                         "run's rows per launch"},
            "predictor": predictor,
            "kernel_us_per_launch": kernel_us,
            "per_token": {"rows_active": rows_active / K, "rows_loaded": fetched / beta / K,
                          "rows_moved": rows_moved / K},
            "cold_start": {"first_token_ms": ms_cold,
                           "host_link_MB_in_warmup": cold_fetched / 1e6,
                           "note": "token 0 starts from an empty cache; the timed region starts after "
                                   f"{Wm} warm-up tokens"},
            "clocks": clock_info,
        }
        out["host_link_whole_token"] = {
            "achieved": fetched / K / (ms_total / K) / 1e6, "peak": link_peak, "unit": "GB/s",
            "frac": fetched / K / (ms_total / K) / 1e6 / link_peak,
            "what": "bundle bytes fetched per token over the token's time: the share of a token "
                    "during which the host link is busy at its measured peak"}
        if detail and args.cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(cfg, layers, X, args.cpu_seconds,
                                               _gate_setup(args), args.append_first)
    else:
        out = None
    B.lif_graph_destroy(graph)
    for l in layers:
        l.close()
    del exchange, layers, handles, graph, X
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return out


def run_kernel_loop(args):
    """For profilers: W warm-up tokens through the graph, then ONE plain launch of the chosen
    kernel on every layer's lists (layer 0 first).  Prints the rows each launch processes, so a
    captured launch can be related to its algorithmic bytes."""
    import torch
    from paper_2312_11514_b200 import binding as B
    from paper_2312_11514_b200 import runtime as R
    from paper_2312_11514_b200 import workloads as W
    dev = "cuda:0"
    cfg = W.CONFIGS[args.config]
    gate_mode, activation, act_thr = _gate_setup(args)
    layers = R.build_stack(cfg, dev, n_layers=args.layers, gate_mode=gate_mode, activation=activation,
                           activation_threshold=act_thr, append_first=args.append_first)
    handles = [l.handle for l in layers]
    for item in args.tune:
        key, value = item.split("=")
        for h in handles:
            B.lif_set_tuning(h, getattr(B, "TUNE_" + key.upper()), int(value))
    L, S, d = len(layers), cfg.n_streams, cfg.d_model
    X = _inputs(cfg, args.warmup, dev, W)
    Y = torch.empty(L, S, d, dtype=torch.float32, device=dev)
    dev_x = torch.empty(S, d, dtype=torch.float16, device=dev)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    graph = B.lif_graph_capture(handles, dev_x, Y, sc, sf)
    for t in range(args.warmup):
        with torch.cuda.stream(sc):
            dev_x.copy_(X[t], non_blocking=True)
        B.lif_graph_launch(graph, sc)
    torch.cuda.synchronize()
    cnt = {"ffn_active": B.CNT_N_ACTIVE, "ffn_hits": B.CNT_N_HITS, "ffn_new": B.CNT_N_LOAD,
           "fetch": B.CNT_N_LOAD, "ffn_api": B.CNT_N_ACTIVE}.get(args.kernel_loop)
    rows = [int(l.counts[cnt]) for l in layers] if cnt is not None else None
    for l in range(L):
        if args.kernel_loop == "ffn_api":     # lif_sparse_ffn over the active rows, any stream count
            B.lif_sparse_ffn(handles[l], dev_x, layers[l]._view("active_slots", cfg.d_ff),
                             layers[l].counts[B.CNT_N_ACTIVE:], Y[l], sc)
        else:
            B.lif_profile_launch(handles[l], B.KERNELS.index(args.kernel_loop), dev_x, Y[l], sc)
    torch.cuda.synchronize()
    print(json.dumps({"kernel": args.kernel_loop, "layers": L, "warmup_tokens": args.warmup,
                      "rows_per_launch": rows,
                      "bundle_bytes": (3 if gate_mode == 1 else 2) * d * 2}), flush=True)
    B.lif_graph_destroy(graph)
    for l in layers:
        l.close()


def run_sweep_k(args):
    """Memory-latency trade-off (the paper's Section 4 figure of latency against the share of
    the model kept in memory): one JSON line per window size k with tokens/s, the share of
    the FFN resident in HBM and the bytes fetched per token."""
    import torch
    from paper_2312_11514_b200 import binding as B
    from paper_2312_11514_b200 import runtime as R
    from paper_2312_11514_b200 import workloads as W
    dev = "cuda:0"
    base = W.CONFIGS[args.config]
    K, Wm = args.steps, args.warmup
    for k in [int(v) for v in args.sweep_k.split(",")]:
        cfg = base.scaled(window_k=k)
        # small windows see the step-to-step swings of the active set undamped: wide margin
        layers = R.build_stack(cfg, dev, n_layers=args.layers, capacity_margin=40.0)
        handles = [l.handle for l in layers]
        L, S, d = len(layers), cfg.n_streams, cfg.d_model
        X = _inputs(cfg, Wm + K, dev, W)
        Y = torch.empty(L, S, d, dtype=torch.float32, device=dev)
        dev_x = torch.empty(S, d, dtype=torch.float16, device=dev)
        sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()
        graph = B.lif_graph_capture(handles, dev_x, Y, sc, sf)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for t in range(Wm + K):
            if t == Wm:
                torch.cuda.synchronize()
                s0 = [B.lif_get_stats(h) for h in handles]
                e0.record(sc)
            with torch.cuda.stream(sc):
                dev_x.copy_(X[t], non_blocking=True)
            B.lif_graph_launch(graph, sc)
        e1.record(sc)
        torch.cuda.synchronize()
        s1 = [B.lif_get_stats(h) for h in handles]
        assert all(s.status == B.LIF_OK for s in s1), [B.status_str(s.status) for s in s1]
        ms = e0.elapsed_time(e1)
        fetched = sum(b.bytes_fetched - a.bytes_fetched for a, b in zip(s0, s1))
        cached = sum(b.rows_cached - a.rows_cached for a, b in zip(s0, s1)) / (K * L)
        print(json.dumps({"window_k": k, "tokens_per_s": K / (ms / 1e3), "ms_per_token": ms / K,
                          "ffn_share_resident": cached / cfg.d_ff,
                          "new_share_per_token": fetched / K / L / cfg.bundle_bytes / cfg.d_ff,
                          "host_link_MB_per_token": fetched / K / 1e6, "layers": L,
                          "config": cfg.name}), flush=True)
        B.lif_graph_destroy(graph)
        for l in layers:
            l.close()
        del layers, graph
        torch.cuda.empty_cache()


# ------------------------------------------------------------------------------ CPU oracle
def _oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def _oracle_layers(cfg, tensors, O, gate=(0, 0, 0.0), append_first=False):
    import numpy as np
    out = []
    for w, cap in tensors:
        out.append(dict(A=w["A"].cpu().numpy().astype(np.float64), B=w["B"].cpu().numpy().astype(np.float64),
                        c=w["c"].cpu().numpy().astype(np.float64), bundles=w["bundles"].cpu().numpy(),
                        bias_up=w["bias_up"].cpu().numpy(),
                        gate=w["gate"].cpu().numpy() if gate[0] == 2 else None,
                        cache=O.NeuronCache(cfg.d_model, cfg.d_ff, cap, cfg.window_k,
                                            n_vec=3 if gate[0] == 1 else 2,
                                            append_first=bool(append_first))))
    return out


def _oracle_token(ol, x_np, O, gate=(0, 0, 0.0)):
    gm, act, thr = gate
    for w in ol:
        if gm == 2:
            O.decode_step_gate_predictor(w["cache"], x_np, w["gate"], w["bias_up"], w["bundles"],
                                         activation=act, threshold=thr)
        else:
            O.decode_step(w["cache"], x_np, w["A"], w["B"], w["c"], 0.0, w["bundles"], w["bias_up"],
                          activation=act, threshold=thr, gated=gm == 1)


def cpu_baseline(cfg, layers, X, seconds, gate=(0, 0, 0.0), append_first=False):
    """The oracle, as it stands, on a bounded sample of the same workload: EVERY layer of the
    stack (a few layers alone stay in the host caches and run almost twice as fast per layer),
    as many tokens as fit about `seconds` of CPU time after window_k + 1 warm-up tokens."""
    from oracle import lif_oracle as O
    tensors = [({"A": l.keep["pred_A"], "B": l.keep["pred_B"], "c": l.keep["pred_c"],
                 "bundles": l.keep["host_bundles"], "bias_up": l.keep["bias_up"],
                 "gate": l.keep["gate"]}, l.capacity)
               for l in layers]
    ol = _oracle_layers(cfg, tensors, O, gate, append_first)
    xs = X.cpu().numpy()
    warm = max(1, min(cfg.window_k + 1, xs.shape[0] - 1))
    for t in range(warm):
        _oracle_token(ol, xs[t], O, gate)
    t0 = time.perf_counter()
    done = 0
    for t in range(warm, xs.shape[0]):
        _oracle_token(ol, xs[t], O, gate)
        done += 1
        if time.perf_counter() - t0 > seconds:
            break
    dt = time.perf_counter() - t0
    return {"value": done / dt, "unit": UNIT, "cores": _oracle_threads(), "kind": "oracle",
            "sample": f"all {len(layers)} layers, tokens {warm}..{warm + done - 1} after {warm} warm-up "
                      f"tokens ({dt:.1f} s of CPU time)"}


def run_reference(args):
    """The CPU oracle as the reference arm: one step = one token through every layer."""
    if int(os.environ.get("RANK", 0)) != 0:
        return
    import torch
    from oracle import lif_oracle as O
    from paper_2312_11514_b200 import workloads as W
    cfg = W.CONFIGS[args.config]
    gate = _gate_setup(args)
    gen = "cuda:0" if torch.cuda.is_available() else "cpu"
    mk = lambda l: W.make_layer(cfg, l, device=gen, gate_mode=gate[0], act_threshold=gate[2])
    L = args.layers or cfg.n_layers
    if not args.layers:
        # bound the run: time one layer-step, then keep as many layers as fit ~2 minutes
        w0 = {k: v.cpu() for k, v in mk(0).items()}
        probe = _oracle_layers(cfg, [(w0, W.window_capacity(cfg, w0["p"]))], O, gate, args.append_first)
        x0 = _inputs(cfg, 2, gen, W).cpu().numpy()
        _oracle_token(probe, x0[0], O, gate)
        t0 = time.perf_counter()
        _oracle_token(probe, x0[1], O, gate)
        per = max(time.perf_counter() - t0, 1e-4)
        L = max(1, min(cfg.n_layers, int(120.0 / ((args.steps + args.warmup) * per))))
        del probe, w0
    tensors = []
    for l in range(L):
        w = {k: v.cpu() for k, v in mk(l).items()}
        tensors.append((w, W.window_capacity(cfg, w["p"])))
    ol = _oracle_layers(cfg, tensors, O, gate, args.append_first)
    K, Wm = args.steps, args.warmup
    xs = _inputs(cfg, Wm + K, gen, W).cpu().numpy()
    for t in range(Wm):
        _oracle_token(ol, xs[t], O, gate)
    t0 = time.perf_counter()
    for t in range(Wm, Wm + K):
        _oracle_token(ol, xs[t], O, gate)
    dt = time.perf_counter() - t0
    v = K / dt * (cfg.n_layers / L)
    cores = _oracle_threads()
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
        "steps": K, "warmup": Wm, "ms_per_step": dt / K * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_string(cfg, cfg.n_layers if not args.layers else L, args.gate,
                                               gate[0], gate[2]),
                   "arm": "CPU oracle (numpy, float64)" + ("" if L == (args.layers or cfg.n_layers) else
                          f": {L} of {cfg.n_layers} layers timed, tokens/s scaled by layers")},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{L} of {cfg.n_layers} layers, every timed token"},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def run_file_store(args):
    """The bundle store in files (the paper's storage tier: reader threads, one read per bundle,
    uncached where the file system allows) instead of pinned host memory: one JSON line per
    thread count with tokens/s, the bytes read per token and the rate the reads reached.  The
    loads are managed on the host, so every layer-step synchronises twice; compare with the same
    --layers through the default (pinned-memory) path."""
    import numpy as np
    import torch
    from paper_2312_11514_b200 import binding as B
    from paper_2312_11514_b200 import runtime as R
    from paper_2312_11514_b200 import workloads as W
    dev = "cuda:0"
    torch.cuda.set_device(0)
    cfg = W.CONFIGS[args.config]
    L = args.layers or min(cfg.n_layers, 8)
    S, d = cfg.n_streams, cfg.d_model
    K, Wm = args.steps, args.warmup
    os.makedirs(args.store_dir, exist_ok=True)
    layers, paths = [], []
    for l in range(L):
        full = R.pinned_store(cfg.d_ff, d)
        w = W.make_layer(cfg, l, device=dev, bundles_out=full)
        path = os.path.join(args.store_dir, f"lif_bundles_{cfg.name}_{l}.bin")
        with open(path, "wb") as f:
            full.numpy().tofile(f)
            f.flush()
            os.fsync(f.fileno())
        paths.append(path)
        cap = min(cfg.d_ff, W.window_capacity(cfg, w["p"]))
        staging = torch.zeros(cap, 2 * d, dtype=torch.float16).pin_memory()
        to = lambda t: t.to(dev).contiguous()
        layers.append(R.Layer(d_model=d, d_ff=cfg.d_ff, rank=cfg.rank, window_k=cfg.window_k, capacity=cap,
                              host_bundles=staging, pred_A=to(w["A"]), pred_B=to(w["B"]), pred_c=to(w["c"]),
                              bias_up=to(w["bias_up"]), n_streams=S, append_first=args.append_first,
                              staging_rows=cap, device=dev))
        del full, w
    X = _inputs(cfg, Wm + K, dev, W)
    Y = torch.empty(L, S, d, dtype=torch.float32, device=dev)
    sc = torch.cuda.Stream()
    try:
        for n_threads in [int(v) for v in args.store_threads.split(",")]:
            stores = [B.lif_store_open(p, cfg.d_ff, cfg.bundle_bytes, n_threads, not args.store_cached)
                      for p in paths]
            for l in layers:
                B.lif_reset(l.handle, sc)
            torch.cuda.synchronize()
            t0 = None
            for t in range(Wm + K):
                if t == Wm:
                    s0 = [B.lif_store_get_stats(s) for s in stores]
                    t0 = time.perf_counter()
                for l in range(L):
                    B.lif_decode_step_store(layers[l].handle, stores[l], X[t], Y[l], sc)
            dt = time.perf_counter() - t0
            s1 = [B.lif_store_get_stats(s) for s in stores]
            req = sum(b.bytes_requested - a.bytes_requested for a, b in zip(s0, s1))
            got = sum(b.bytes_read - a.bytes_read for a, b in zip(s0, s1))
            secs = sum(b.seconds_reading - a.seconds_reading for a, b in zip(s0, s1))
            reads = sum(b.reads - a.reads for a, b in zip(s0, s1))
            assert all(B.lif_get_stats(l.handle).status == B.LIF_OK for l in layers)
            print(json.dumps({
                "mode": "file_store", "config": cfg.name, "layers": L, "steps": K, "warmup": Wm,
                "reader_threads": n_threads, "direct_io": bool(s1[0].direct_io),
                "tokens_per_s_these_layers": K / dt, "ms_per_layer_step": dt / (K * L) * 1e3,
                "bundle_MB_per_token": req / K / 1e6, "bytes_read_over_requested": got / max(req, 1),
                "read_GBs_while_reading": req / max(secs, 1e-9) / 1e9,
                "read_calls_per_s_while_reading": reads / max(secs, 1e-9),
                "share_of_time_in_reads": secs / dt, "bundle_bytes": cfg.bundle_bytes,
                "store_dir": args.store_dir}), flush=True)
            for s in stores:
                B.lif_store_close(s)
    finally:
        for l in layers:
            l.close()
        for p in paths:
            os.remove(p)


def run_stub(args):
    """Stand-in arm without a device, for testing the multi-rank plumbing on CPU: every rank
    'decodes' its K tokens by sleeping (1 + rank) ms per token, the ranks meet at a barrier, the
    slowest rank's time is taken, and rank 0 prints the line with the whole-job rate."""
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    for _ in range(args.warmup):
        time.sleep(0.001)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.001 * (1 + rank))
    ms = (time.perf_counter() - t0) * 1e3
    if world > 1:
        dist.barrier()
    ms_slowest = max_over_ranks(ms, world, "cpu")
    if rank == 0:
        print(json.dumps({"impl": "stub", "metric": METRIC, "unit": UNIT, "n_gpus": world,
                          "value": whole_job_tokens_per_s(args.steps, world, ms_slowest),
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_slowest / args.steps,
                          "higher_is_better": True, "scaling": "weak", "data": "none",
                          "config": {"workload": "stub", "parallelism": "independent sequence per rank"}}),
              flush=True)
    if world > 1:
        dist.destroy_process_group()


def launch_ranks(args):
    """`--gpus N` with N > 1 outside torchrun: start N ranks of this script on this node (one per
    GPU, rendezvous on 127.0.0.1) and pass their output through.  Returns the exit code."""
    import socket
    if args.impl == "ours":
        import torch
        have = torch.cuda.device_count() if torch.cuda.is_available() else 0
        if have < args.gpus:
            print(f"bench.py: --gpus {args.gpus} needs {args.gpus} CUDA devices on this node, found {have}",
                  file=sys.stderr)
            return 2
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")            # the communicator's set-up goes to stderr
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def run_floors(args):
    """Reference points that the kernels are judged against, measured with calls the library
    exports: the host link (copy engine, and a kernel reading mapped host memory), and what a
    kernel that does nothing but read a few MB of HBM achieves per launch when it is launched the
    way the decode step launches its kernels (a graph of dependent launches, L2-cold)."""
    import torch
    from paper_2312_11514_b200 import binding as B
    dev = "cuda:0"
    torch.cuda.set_device(0)
    st = torch.cuda.Stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    out = {"mode": "floors", "hbm_peak_GBs": _peaks()[0], "hbm_peak_kind": _peaks()[1]}

    def timed(fn, reps):
        with torch.cuda.stream(st):
            fn()
            e0.record(st)
            for _ in range(reps):
                fn()
            e1.record(st)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / reps          # us

    # ---- host link
    nb = 1 << 30
    hbuf = torch.empty(nb, dtype=torch.uint8, pin_memory=True)
    dbuf = torch.empty(nb, dtype=torch.uint8, device=dev)
    best = min(timed(lambda: dbuf.copy_(hbuf, non_blocking=True), 1) for _ in range(5))
    link = {"cudaMemcpyAsync_1GiB_GBs": nb / best / 1e3}
    best = min(timed(lambda: B.lif_probe_host_read(hbuf, dbuf, nb, 16384, st), 1) for _ in range(3))
    link["kernel_read_1GiB_16KiB_chunks_GBs"] = nb / best / 1e3
    # the same host memory through bulk copies into shared memory (the probe takes any global
    # address: mapped host memory is one), 16 KiB per copy, 1 and 4 CTAs per SM
    sink0 = torch.zeros(16, dtype=torch.uint8, device=dev)
    tmo0 = torch.zeros(1, dtype=torch.int32, device=dev)
    for ctas, stages in ((1, 4), (4, 3)):
        best = min(timed(lambda: B.lif_probe_bulk_ring(hbuf, nb, 16384, stages, 1, ctas, 0, sink0, tmo0, st), 1)
                   for _ in range(3))
        link[f"bulk_copies_1GiB_16KiB_{ctas}cta_per_sm_GBs"] = nb / best / 1e3
    link["bulk_copy_waits_that_ran_out"] = int(tmo0.item())
    for mb in (1, 2, 4, 8):
        n = mb << 20
        offs = [(i * 97 % 509) * (2 << 20) for i in range(24)]      # different regions: no reuse
        it = iter(range(10 ** 9))
        us = timed(lambda: B.lif_probe_host_read(hbuf[offs[next(it) % 24]:], dbuf, n, 16384, st), 24)
        it = iter(range(10 ** 9))
        us_cp = timed(lambda: dbuf[:n].copy_(hbuf[offs[next(it) % 24]:][:n], non_blocking=True), 24)
        link[f"{mb}MiB_per_launch"] = {"kernel_read_us": us, "kernel_read_GBs": n / us / 1e3,
                                       "cudaMemcpyAsync_us": us_cp, "cudaMemcpyAsync_GBs": n / us_cp / 1e3}
    out["host_link"] = link
    del hbuf

    # ---- HBM streaming read per launch, launched like the decode step's kernels
    pool = torch.empty(2 << 30, dtype=torch.uint8, device=dev)       # 2 GiB: every launch is L2-cold
    pool.zero_()
    sink = torch.zeros(16, dtype=torch.uint8, device=dev)
    reads = {}
    for mb in (1, 2, 4, 6, 8, 16, 64):
        n = mb << 20
        n_regions = min(64, (2 << 30) // n)
        for ctas in (1, 2, 4):
            for pdl in (1, 0):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=st):
                    for i in range(32):
                        off = (i * 37 % n_regions) * n
                        B.lif_probe_device_read(pool[off:], n, sink, ctas, bool(pdl), st)
                us = timed(g.replay, 10) / 32
                reads[f"{mb}MiB_{ctas}cta_per_sm_{'dependent' if pdl else 'plain'}"] = {
                    "us_per_launch": us, "GBs": n / us / 1e3, "frac_of_hbm_peak": n / us / 1e3 / out["hbm_peak_GBs"]}
                del g
    out["hbm_read_per_launch_in_graph"] = reads
    # ---- streaming through a shared-memory ring of bulk copies (how the FFN kernels bring rows in)
    rings = {}
    tmo = torch.zeros(1, dtype=torch.int32, device=dev)
    nbytes = 160 << 20
    for chunk, stages, group, ctas, every in (
            (3584, 48, 16, 1, 0), (7168, 32, 16, 1, 0), (14336, 16, 8, 1, 0), (14336, 12, 4, 1, 0),
            (28672, 8, 4, 1, 0), (7168, 14, 7, 2, 0), (3584, 14, 7, 4, 0), (16384, 3, 1, 4, 0),
            (3584, 48, 16, 1, 2), (7168, 32, 16, 1, 2), (3584, 48, 16, 1, 1), (7168, 32, 16, 1, 1),
            (7168, 28, 14, 1, 2), (14336, 16, 8, 1, 2)):
        it = iter(range(10 ** 9))
        us = min(timed(lambda: B.lif_probe_bulk_ring(pool[(next(it) % 12) * nbytes:], nbytes, chunk, stages,
                                                     group, ctas, every, sink, tmo, st), 1)
                 for _ in range(5))
        how = "bulk copies" if every == 0 else ("16-byte async copies" if every == 1 else
                                                f"every {every}nd stage by 16-byte async copies")
        rings[f"{chunk}B_x{stages}_refill{group}_{ctas}cta_per_sm_{how}"] = {
            "us": us, "GBs": nbytes / us / 1e3, "frac_of_hbm_peak": nbytes / us / 1e3 / out["hbm_peak_GBs"]}
    assert int(tmo.item()) == 0, "a ring probe's wait ran out"
    out["bulk_copy_ring_160MiB"] = rings
    # the same kernel launched on a stream, one launch at a time (what a graph saves)
    n = 8 << 20
    it = iter(range(10 ** 9))
    us = timed(lambda: B.lif_probe_device_read(pool[(next(it) % 64) * n:], n, sink, 2, True, st), 64)
    out["hbm_read_8MiB_stream_launches_us"] = us
    print(json.dumps(out), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "stub"],
                    help="'stub': no device, for testing the multi-rank plumbing on CPU")
    ap.add_argument("--config", default="opt6p7b")
    ap.add_argument("--layers", type=int, default=None, help="use only the first N layers")
    ap.add_argument("--gate", default="none", choices=sorted(GATE_MODES),
                    help="gated FFN: gate row inside the bundle, or resident gate projection as the "
                         "predictor (use with --config llama2_7b)")
    ap.add_argument("--act-threshold", type=float, default=0.05, help="FATReLU threshold of gated runs")
    ap.add_argument("--append-first", type=int, default=1, choices=[0, 1],
                    help="1: stack the new neurons before deleting, so their bundles go straight into "
                         "freed rows; 0: the order of Section 3.3 as written (same cached set and outputs)")
    ap.add_argument("--shard", default="sequences", choices=["sequences", "neurons"],
                    help="N > 1: 'sequences' = one independent sequence and stack per GPU (default); "
                         "'neurons' = one sequence, every layer's neurons split over the GPUs, partial "
                         "outputs all-reduced after every layer")
    ap.add_argument("--exchange", default="nccl", choices=["nccl", "peer"],
                    help="--shard neurons: sum the partial outputs with an NCCL all-reduce, or with "
                         "lif_sum_peer_outputs reading the peers' partials from peer-mapped memory")
    ap.add_argument("--no-cpu-baseline", dest="cpu_baseline", action="store_false")
    ap.add_argument("--cpu-seconds", type=float, default=12.0,
                    help="CPU time the oracle baseline may take after its warm-up tokens")
    ap.add_argument("--no-other-configs", dest="other_configs", action="store_false",
                    help="leave out the reduced-length runs of the other configurations")
    ap.add_argument("--tune", action="append", default=[], metavar="KNOB=VALUE",
                    help="set a LIF_TUNE_* knob on every layer before capture, e.g. "
                         "--tune batched_up_whole_rows=0 (repeatable)")
    ap.add_argument("--store", default="pinned", choices=["pinned", "file"],
                    help="'file': the bundles of --layers layers (default 8) are written to files under "
                         "--store-dir and read by reader threads (lif_decode_step_store)")
    ap.add_argument("--store-dir", default="/tmp/lif_store")
    ap.add_argument("--store-threads", default="32", help="comma-separated reader thread counts")
    ap.add_argument("--store-cached", action="store_true", help="read through the page cache (no O_DIRECT)")
    ap.add_argument("--floors", action="store_true",
                    help="measure the reference points (host link, HBM read per launch) and exit")
    ap.add_argument("--kernel-loop", default=None,
                    help="profiling aid: after the warm-up tokens launch this kernel once per layer "
                         "(predict_z, predict_scores, fetch, ffn_active, ffn_hits, ffn_new, ffn_sum; "
                         "ffn_api = lif_sparse_ffn over the active rows, for any number of streams)")
    ap.add_argument("--sweep-k", default=None,
                    help="comma-separated window sizes: memory-latency trade-off, one line per k")
    args = ap.parse_args()
    if args.warmup < 3:     # fewer than 3 warm-up steps would make the timing invalid: do 3
        print(f"bench.py: --warmup {args.warmup} raised to 3", file=sys.stderr)
        args.warmup = 3
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl != "reference":
        sys.exit(launch_ranks(args))
    if args.impl == "stub":
        run_stub(args)
    elif args.floors:
        run_floors(args)
    elif args.store == "file":
        run_file_store(args)
    elif args.sweep_k:
        run_sweep_k(args)
    elif args.kernel_loop:
        run_kernel_loop(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        if int(os.environ.get("WORLD_SIZE", 1)) > 1:
            args.cpu_baseline = False
        run_ours(args)


if __name__ == "__main__":
    main()
