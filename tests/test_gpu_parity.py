"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs — scores and outputs within 2e-3, index lists and window state bit-exact."""
import numpy as np
import pytest
import torch

from oracle import lif_oracle as O
from paper_2312_11514_b200 import binding as B
from paper_2312_11514_b200 import runtime as R
from paper_2312_11514_b200 import workloads as W

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run_staged(cfg, layer_idx, steps, **kw):
    whole = kw.get("ffn_mode", 0) == 1
    gpu, ora = P.make_layer_pair(cfg, layer_idx, **kw)
    X = W.make_inputs(cfg, device=DEV)
    bufs = P.make_bufs(gpu)
    stats = [P.staged_step(gpu, ora, X[t], bufs, whole_cache=whole) for t in range(steps)]
    st = B.lif_get_stats(gpu.handle)
    assert st.status == B.LIF_OK
    assert st.bytes_fetched == ora.cache.bytes_fetched == sum(s["n_load"] for s in stats) * cfg.bundle_bytes
    assert st.rows_moved == ora.cache.rows_moved
    gpu.close()
    return stats


@pytest.mark.parametrize("layer_idx", [0, 1])
def test_tiny_config_every_stage_every_step(layer_idx):
    cfg = W.CONFIGS["tiny"]
    stats = _run_staged(cfg, layer_idx, cfg.steps, b_down=(layer_idx == 1))
    assert stats[0]["n_load"] == stats[0]["n_active"] > 0            # cold start
    assert sum(s["n_evict"] for s in stats) > 0


@pytest.mark.parametrize("d,F,r,k,S", [
    (264, 1000, 24, 3, 1),      # ragged: nothing a multiple of the tile sizes
    (328, 2056, 8, 1, 1),       # window of one token, smallest rank
    (4544, 1280, 128, 2, 1),    # Falcon row length (71 x 64), several rows per CTA round
    (512, 4096, 40, 4, 3),      # three streams
    (256, 1536, 16, 2, 8),      # eight streams
])
def test_ragged_shapes_and_streams(d, F, r, k, S):
    cfg = W.LifConfig("ragged", 1, d, F, r, k, S, 12, 0.06, 1.0, 0.8, 0.6, 11)
    stats = _run_staged(cfg, 0, cfg.steps, b_down=True)
    assert sum(s["n_evict"] for s in stats) > 0


def test_whole_cache_mode_and_more_rows_than_stages():
    # mode 1 runs the FFN over every cached row (matrix[:num_used]); with ~40% firing the
    # cache holds far more rows than CTAs x stages of a tiny grid would cover in one round
    cfg = W.LifConfig("dense", 1, 2048, 8192, 32, 3, 1, 6, 0.40, 0.5, 0.8, 0.6, 12)
    stats = _run_staged(cfg, 0, cfg.steps, ffn_mode=1, capacity=8192)
    assert max(s["n_active"] for s in stats) > 148 * 16


def test_threshold_extremes():
    cfg = W.CONFIGS["tiny"]
    X = W.make_inputs(cfg, device=DEV)
    # theta = +inf: nothing is active, y = b_down
    gpu, ora = P.make_layer_pair(cfg, 0, theta=float("inf"), b_down=True)
    bufs = P.make_bufs(gpu)
    s = P.staged_step(gpu, ora, X[0], bufs)
    assert s["n_active"] == 0
    np.testing.assert_array_equal(bufs["y"].cpu().numpy()[0], ora.b_down.astype(np.float32))
    gpu.close()
    # theta = -inf: every neuron is active; the sparse FFN over all rows is the dense FFN
    gpu, ora = P.make_layer_pair(cfg, 0, theta=float("-inf"), capacity=cfg.d_ff)
    bufs = P.make_bufs(gpu)
    s = P.staged_step(gpu, ora, X[0], bufs)
    assert s["n_active"] == cfg.d_ff == s["n_load"]
    Wb = ora.bundles.astype(np.float64)
    x = X[0, 0].cpu().numpy().astype(np.float64)
    dense = np.maximum(Wb[:, :cfg.d_model] @ x + ora.bias_up.astype(np.float64), 0) @ Wb[:, cfg.d_model:]
    P.assert_y_close(bufs["y"].cpu().numpy().astype(np.float64), dense[None, :])
    s = P.staged_step(gpu, ora, X[1], bufs)
    assert s["n_load"] == 0 and s["n_evict"] == 0
    gpu.close()


def test_capacity_overflow_sets_status_and_leaves_state():
    cfg = W.CONFIGS["tiny"]
    X = W.make_inputs(cfg, device=DEV)
    gpu, ora = P.make_layer_pair(cfg, 0, capacity=64)
    bufs = P.make_bufs(gpu)
    act = torch.arange(0, 40, dtype=torch.int32, device=DEV)
    n = torch.tensor([40], dtype=torch.int32, device=DEV)
    B.lif_window_update(gpu.handle, act, n)
    B.lif_fetch_bundles(gpu.handle)
    before = gpu.lists()
    assert before["status"] == B.LIF_OK and before["num_used"] == 40
    act2 = torch.arange(100, 130, dtype=torch.int32, device=DEV)      # 40 kept + 30 new > 64
    n2 = torch.tensor([30], dtype=torch.int32, device=DEV)
    B.lif_window_update(gpu.handle, act2, n2)
    B.lif_fetch_bundles(gpu.handle)
    B.lif_sparse_ffn(gpu.handle, X[0], gpu._view("active_slots", cfg.d_ff), gpu.counts[B.CNT_N_ACTIVE:], bufs["y"])
    after = gpu.lists()
    assert after["status"] == B.LIF_ERR_CAPACITY
    assert B.lif_get_stats(gpu.handle).status == B.LIF_ERR_CAPACITY
    for key in ("pointers", "slot_of", "last_active"):
        np.testing.assert_array_equal(before[key], after[key])
    assert (after["num_used"], after["step"]) == (before["num_used"], before["step"])
    assert len(after["load_ids"]) == 0 and len(after["active_slots"]) == 0
    assert (bufs["y"].cpu().numpy() == 0).all()                       # nothing active, no b_down
    # out-of-range neuron id: refused the same way
    B.lif_clear_status(gpu.handle)
    bad = torch.tensor([5, 5000], dtype=torch.int32, device=DEV)
    B.lif_window_update(gpu.handle, bad, torch.tensor([2], dtype=torch.int32, device=DEV))
    assert gpu.lists()["status"] == B.LIF_ERR_INVALID_ARG
    # after clearing, a fitting step proceeds and matches the oracle
    B.lif_clear_status(gpu.handle)
    ora.cache.window_update(np.arange(40, dtype=np.int32))
    act3 = torch.arange(30, 50, dtype=torch.int32, device=DEV)
    B.lif_window_update(gpu.handle, act3, torch.tensor([20], dtype=torch.int32, device=DEV))
    ref = ora.cache.window_update(np.arange(30, 50, dtype=np.int32))
    P.compare_lists_and_state(gpu, ora, ref)
    gpu.close()


def test_reset_gives_cold_cache_and_runs_are_reproducible():
    cfg = W.CONFIGS["tiny"]
    X = W.make_inputs(cfg, device=DEV)
    gpu, ora = P.make_layer_pair(cfg, 0)
    y = torch.empty(8, cfg.n_streams, cfg.d_model, dtype=torch.float32, device=DEV)
    runs = []
    for _ in range(2):
        B.lif_reset(gpu.handle)
        acts = []
        for t in range(8):
            B.lif_decode_step(gpu.handle, X[t], y[t])
            acts.append(gpu.lists()["active_idx"].copy())
        runs.append((acts, y.cpu().numpy().copy(), gpu.lists()))
    for a, b in zip(runs[0][0], runs[1][0]):
        np.testing.assert_array_equal(a, b)
    assert np.array_equal(runs[0][1].view(np.uint32), runs[1][1].view(np.uint32))     # bitwise
    np.testing.assert_array_equal(runs[0][2]["pointers"], runs[1][2]["pointers"])
    assert runs[1][2]["step"] == 8
    gpu.close()


@pytest.mark.parametrize("two_streams,pdl,split,ffn_mode,fused", [
    (False, 1, 1, 0, 1), (True, 1, 1, 0, 1), (True, 0, 1, 0, 1), (True, 1, 0, 0, 1), (True, 0, 0, 0, 0),
    (True, 1, 1, 1, 1), (False, 1, 0, 1, 0), (True, 1, 1, 0, 0)])
def test_decode_step_matches_oracle_decode_step(two_streams, pdl, split, ffn_mode, fused):
    cfg = W.CONFIGS["tiny"]
    X = W.make_inputs(cfg, device=DEV)
    gpu, ora = P.make_layer_pair(cfg, 1, b_down=True, ffn_mode=ffn_mode)
    B.lif_set_tuning(gpu.handle, B.TUNE_DEPENDENT_LAUNCH, pdl)
    B.lif_set_tuning(gpu.handle, B.TUNE_SPLIT_FFN, split)
    B.lif_set_tuning(gpu.handle, B.TUNE_FUSED_PLAN, fused)
    y = torch.empty(cfg.n_streams, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = (torch.cuda.Stream(), torch.cuda.Stream()) if two_streams else (None, None)
    if sc is not None:
        sc.wait_stream(torch.cuda.current_stream())
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        g = gpu.lists()
        x_np = X[t].cpu().numpy()
        logits, act, lists, ref_y = O.decode_step(ora.cache, x_np, ora.A, ora.B, ora.c, ora.theta,
                                                  ora.bundles, ora.bias_up, ora.b_down,
                                                  whole_cache=(ffn_mode == 1), act=g["active_idx"])
        P.assert_mask_borderline(g["active_idx"], logits, ora.theta)
        P.compare_lists_and_state(gpu, ora, lists)
        P.compare_cache_rows(gpu, ora)
        P.assert_y_close(y.cpu().numpy().astype(np.float64), ref_y)
    gpu.close()


def test_decode_token_host_matches_per_layer_decode_steps():
    cfg = W.CONFIGS["tiny"]
    X = W.make_inputs(cfg, device=DEV)
    a = R.build_stack(cfg, DEV)
    b = R.build_stack(cfg, DEV)
    L, S, d = cfg.n_layers, cfg.n_streams, cfg.d_model
    host_x = torch.empty(S, d, dtype=torch.float16, pin_memory=True)
    host_y = torch.empty(L, S, d, dtype=torch.float32, pin_memory=True)
    dev_x = torch.empty(S, d, dtype=torch.float16, device=DEV)
    dev_y = torch.empty(L, S, d, dtype=torch.float32, device=DEV)
    y_ref = torch.empty(L, S, d, dtype=torch.float32, device=DEV)
    sc, sf, sc2, sf2 = (torch.cuda.Stream() for _ in range(4))
    torch.cuda.synchronize()
    for t in range(10):
        host_x.copy_(X[t])
        B.lif_decode_token_host([l.handle for l in a], host_x, dev_x, dev_y, host_y, sc, sf)
        for l in range(L):
            B.lif_decode_step(b[l].handle, X[t], y_ref[l], sc2, sf2)
        torch.cuda.synchronize()
        assert torch.equal(host_y, y_ref.cpu())
    for l in range(L):
        assert B.lif_get_stats(a[l].handle).bytes_fetched == B.lif_get_stats(b[l].handle).bytes_fetched > 0
    for l in a + b:
        l.close()


@pytest.mark.parametrize("append_first", [0, 1])
def test_graph_replay_matches_direct_decode_steps_bitwise(append_first):
    cfg = W.CONFIGS["tiny"]
    X = W.make_inputs(cfg, device=DEV)
    a = R.build_stack(cfg, DEV, append_first=append_first)
    b = R.build_stack(cfg, DEV, append_first=append_first)
    L, S, d = cfg.n_layers, cfg.n_streams, cfg.d_model
    dev_x = torch.empty(S, d, dtype=torch.float16, device=DEV)
    y_g = torch.zeros(L, S, d, dtype=torch.float32, device=DEV)
    y_d = torch.zeros(L, S, d, dtype=torch.float32, device=DEV)
    host_x = torch.empty(S, d, dtype=torch.float16, pin_memory=True)
    host_y = torch.empty(L, S, d, dtype=torch.float32, pin_memory=True)
    sc, sf, sc2, sf2 = (torch.cuda.Stream() for _ in range(4))
    torch.cuda.synchronize()
    g = B.lif_graph_capture([l.handle for l in a], dev_x, y_g, sc, sf)
    assert all(l.lists()["step"] == 0 for l in a)                     # capture ran nothing
    for t in range(cfg.steps):
        if t % 2 == 0:
            with torch.cuda.stream(sc):
                dev_x.copy_(X[t])
            B.lif_graph_launch(g, sc)
            torch.cuda.synchronize()
            got = y_g.cpu()
        else:
            host_x.copy_(X[t])
            B.lif_graph_launch_host(g, host_x, host_y, sc)
            got = host_y.clone()
        for l in range(L):
            B.lif_decode_step(b[l].handle, X[t], y_d[l], sc2, sf2)
        torch.cuda.synchronize()
        assert torch.equal(got, y_d.cpu()), t
    for la, lb in zip(a, b):
        ga, gb = la.lists(), lb.lists()
        for key in ("pointers", "slot_of", "last_active", "active_idx", "load_ids"):
            np.testing.assert_array_equal(ga[key], gb[key])
        assert ga["step"] == cfg.steps and ga["status"] == B.LIF_OK
    B.lif_graph_destroy(g)
    for l in a + b:
        l.close()


def test_decode_step_with_dense_mask_and_large_cache():
    # ~40 % of the neurons fire: mask words hold more active neurons than the fused window
    # update keeps in registers, and the cache outgrows its per-thread slots, so the kernel
    # must hand over to its general path inside the same launch
    cfg = W.LifConfig("dense", 1, 512, 16384, 32, 2, 1, 5, 0.40, 0.5, 0.8, 0.6, 13)
    X = W.make_inputs(cfg, device=DEV)
    gpu, ora = P.make_layer_pair(cfg, 0, capacity=cfg.d_ff)
    y = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        g = gpu.lists()
        logits, act, lists, ref_y = O.decode_step(ora.cache, X[t].cpu().numpy(), ora.A, ora.B, ora.c,
                                                  0.0, ora.bundles, ora.bias_up, act=g["active_idx"])
        P.assert_mask_borderline(g["active_idx"], logits, 0.0)
        P.compare_lists_and_state(gpu, ora, lists)
        P.compare_cache_rows(gpu, ora)
        P.assert_y_close(y.cpu().numpy().astype(np.float64), ref_y)
    assert g["num_used"] > 4096
    gpu.close()


@pytest.mark.parametrize("activation,thr,S", [(B.ACT_RELU_SQUARED, 0.0, 1), (B.ACT_FATRELU, 0.15, 1),
                                              (B.ACT_RELU_SQUARED, 0.0, 3), (B.ACT_FATRELU, 0.15, 8)])
def test_activation_variants(activation, thr, S):
    # squared ReLU and FATReLU (Appendix C: Persimmon 8B, Llama 2) through the staged entry
    # points; a high firing rate so that many neurons pass the non-linearity
    cfg = W.LifConfig("act", 1, 512, 2048, 16, 3, S, 6, 0.30, 0.5, 0.8, 0.6, 14)
    stats = _run_staged(cfg, 0, cfg.steps, b_down=True, activation=activation, act_threshold=thr,
                        capacity=2048)
    assert min(s["n_active"] for s in stats) > 100


@pytest.mark.parametrize("fused", [0, 1])
def test_memory_budget_shrinks_the_window(fused):
    # Appendix C (Persimmon 8B, Phi-2): a row budget below the natural window union forces
    # the window to shrink on some steps.  fused = 0: staged entry points (general window
    # kernel); fused = 1: lif_decode_step (mask-fed kernel).
    cfg = W.LifConfig("budget", 1, 256, 4096, 16, 5, 1, 24, 0.05, 1.0, 0.5, 0.87, 15)
    budget = 600
    if not fused:
        stats = _run_staged(cfg, 0, cfg.steps, budget_rows=budget, capacity=1024)
        ks = [s["k_eff"] for s in stats]
        assert max(s["num_used"] for s in stats) <= budget
    else:
        gpu, ora = P.make_layer_pair(cfg, 0, budget_rows=budget, capacity=1024)
        X = W.make_inputs(cfg, device=DEV)
        y = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
        sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()
        ks = []
        for t in range(cfg.steps):
            B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
            g = gpu.lists()
            _, _, lists, ref_y = O.decode_step(ora.cache, X[t].cpu().numpy(), ora.A, ora.B, ora.c, 0.0,
                                               ora.bundles, ora.bias_up, act=g["active_idx"])
            P.compare_lists_and_state(gpu, ora, lists)
            P.compare_cache_rows(gpu, ora)
            P.assert_y_close(y.cpu().numpy().astype(np.float64), ref_y)
            assert g["num_used"] <= budget
            ks.append(g["k_eff"])
        gpu.close()
    assert min(ks) < cfg.window_k and max(ks) == cfg.window_k, ks     # shrinks on some steps only


@pytest.mark.parametrize("keep,fused", [(5, 0), (2, 0), (2, 1), (1, 1)])
def test_speculative_multi_token_window(keep, fused):
    # Section 4, speculative decoding: a step verifies lambda + 1 = 5 consecutive tokens; the
    # window keeps the last k tokens ending with token `keep` of the step
    S = 5
    cfg = W.LifConfig("spec", 1, 256, 4096, 16, 3, S, 10, 0.03, 1.0, 0.8, 0.6, 16)
    gpu, ora = P.make_layer_pair(cfg, 0, spec_keep=keep, capacity=2048)
    Xs = W.make_inputs(cfg.scaled(n_streams=1, steps=cfg.steps * S), device=DEV)   # one sequence
    X = Xs.reshape(cfg.steps, S, cfg.d_model).contiguous()                          # S tokens per step
    if not fused:
        bufs = P.make_bufs(gpu)
        stats = [P.staged_step(gpu, ora, X[t], bufs) for t in range(cfg.steps)]
        assert sum(s["n_evict"] for s in stats) > 0
    else:
        y = torch.empty(S, cfg.d_model, dtype=torch.float32, device=DEV)
        sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()
        for t in range(cfg.steps):
            B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
            g = gpu.lists()
            x_np = X[t].cpu().numpy()
            logits = O.predictor_logits(x_np, ora.A, ora.B, ora.c)
            P.assert_mask_borderline(g["active_idx"], logits, 0.0)
            kt = P.keep_tokens_checked(gpu, g["active_idx"], logits, 0.0)
            _, _, lists, ref_y = O.decode_step(ora.cache, x_np, ora.A, ora.B, ora.c, 0.0, ora.bundles,
                                               ora.bias_up, act=g["active_idx"], keep_token=kt, keep=keep)
            P.compare_lists_and_state(gpu, ora, lists)
            P.compare_cache_rows(gpu, ora)
            P.assert_y_close(y.cpu().numpy().astype(np.float64), ref_y)
    assert gpu.lists()["step"] == cfg.steps * keep == ora.cache.t
    gpu.close()


def test_snapshot_restore_resumes_bit_identically():
    cfg = W.CONFIGS["tiny"]
    X = W.make_inputs(cfg, device=DEV)
    gpu, ora = P.make_layer_pair(cfg, 0)
    y = torch.empty(cfg.steps, 1, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    def run(t0, t1):
        out = []
        for t in range(t0, t1):
            B.lif_decode_step(gpu.handle, X[t], y[t], sc, sf)
            out.append(gpu.lists())
        return out, y[t0:t1].cpu().numpy().copy()
    run(0, 10)
    snap = B.lif_snapshot(gpu.handle)
    # read_state agrees with the device views
    ptr = np.empty(gpu.capacity, dtype=np.int32); so = np.empty(cfg.d_ff, dtype=np.int32)
    la = np.empty(cfg.d_ff, dtype=np.int32); nu = np.empty(1, dtype=np.int32)
    B.lif_read_state(gpu.handle, ptr, so, la, nu)
    g = gpu.lists()
    np.testing.assert_array_equal(ptr, g["pointers"]); np.testing.assert_array_equal(so, g["slot_of"])
    np.testing.assert_array_equal(la, g["last_active"]); assert nu[0] == g["num_used"]
    first_lists, first_y = run(10, 20)
    # wreck the device state and cache, then restore and replay
    B.lif_reset(gpu.handle)
    gpu.cache.zero_()
    torch.cuda.synchronize()
    B.lif_restore(gpu.handle, snap)
    assert gpu.lists()["step"] == 10
    again_lists, again_y = run(10, 20)
    assert np.array_equal(first_y.view(np.uint32), again_y.view(np.uint32))
    for a, b in zip(first_lists, again_lists):
        for key in ("active_idx", "load_ids", "evict_ids", "move_src", "active_slots", "pointers", "last_active"):
            np.testing.assert_array_equal(a[key], b[key], err_msg=key)
    # a snapshot whose counters do not fit is refused
    bad = bytearray(snap); bad[B.CNT_NUM_USED * 4:B.CNT_NUM_USED * 4 + 4] = (10 ** 6).to_bytes(4, "little")
    with pytest.raises(B.LifError) as e:
        B.lif_restore(gpu.handle, bytes(bad))
    assert e.value.code == B.LIF_ERR_STATE
    gpu.close()


def test_window_longer_than_the_sequence_never_evicts():
    cfg = W.LifConfig("longwin", 1, 256, 2048, 16, 64, 1, 10, 0.04, 1.0, 0.8, 0.6, 17)
    gpu, ora = P.make_layer_pair(cfg, 0, capacity=2048)
    X = W.make_inputs(cfg, device=DEV)
    bufs = P.make_bufs(gpu)
    stats = [P.staged_step(gpu, ora, X[t], bufs) for t in range(cfg.steps)]
    assert sum(s["n_evict"] for s in stats) == 0 and B.lif_get_stats(gpu.handle).rows_moved == 0
    used = [s["num_used"] for s in stats]
    assert used == sorted(used) and used[-1] > used[0]                # the cache only grows
    gpu.close()


@pytest.mark.parametrize("d,F,k,act,thr,gate_mode,ffn_mode", [
    (256, 1024, 3, B.ACT_RELU, 0.0, 0, 0),
    (264, 1000, 2, B.ACT_FATRELU, 0.1, 0, 0),         # ragged row length
    (8192, 520, 2, B.ACT_RELU_SQUARED, 0.0, 0, 0),    # widest row: four chunks per thread
    (4096, 1408, 2, B.ACT_RELU, 0.0, 0, 1),           # whole-cache FFN
    (512, 2048, 2, B.ACT_FATRELU, 0.05, 2, 0),        # resident gate
    (512, 2048, 2, B.ACT_FATRELU, 0.05, 1, 0),        # bundled gate: falls back to two kernels
])
@pytest.mark.parametrize("fused_fetch", [1, 0])
def test_decode_step_with_and_without_the_fused_fetch(d, F, k, act, thr, gate_mode, ffn_mode, fused_fetch):
    # lif_decode_step either lets the fetch kernel add the new rows' FFN terms or runs the
    # FFN kernel over them afterwards; both must match the oracle
    cfg = W.LifConfig("fusedfetch", 1, d, F, 16, k, 1, 10, 0.08, 1.0, 0.8, 0.6, 31)
    gpu, ora = P.make_layer_pair(cfg, 0, activation=act, act_threshold=thr, gate_mode=gate_mode,
                                 ffn_mode=ffn_mode, b_down=True)
    B.lif_set_tuning(gpu.handle, B.TUNE_FUSED_FETCH_FFN, fused_fetch)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(1, d, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    n_load = n_evict = 0
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        torch.cuda.synchronize()
        x_np = X[t].cpu().numpy()
        if ffn_mode == 0:
            lists = P.check_decode_step(gpu, ora, x_np, y)
        else:
            g = gpu.lists()
            lists = ora.cache.window_update(g["active_idx"])
            ora.cache.insert(lists, ora.bundles, ora.bias_up)
            P.compare_lists_and_state(gpu, ora, lists)
            ref_y, flips = P.ffn_reference(ora, np.arange(ora.cache.num_used), x_np)
            P.assert_y_close(y.cpu().numpy().astype(np.float64), ref_y, flips)
        P.compare_cache_rows(gpu, ora)
        n_load += len(lists["load_ids"]); n_evict += len(lists["evict_ids"])
    assert n_load > 0 and n_evict > 0
    gpu.close()


# ---- append-first order of the cache operations (new neurons stacked, then the deletions) ----
@pytest.mark.parametrize("d,F,r,k,S,fire", [
    (256, 1024, 16, 3, 1, 0.05),
    (264, 1000, 24, 1, 1, 0.08),      # window of one token: as many deletions as arrivals, roughly
    (512, 4096, 40, 4, 3, 0.04),      # three streams
    (2048, 8192, 32, 3, 1, 0.40),     # more than 4096 cached rows: the general window kernel
])
def test_append_first_staged(d, F, r, k, S, fire):
    cfg = W.LifConfig("af", 1, d, F, r, k, S, 12, fire, 1.0, 0.8, 0.6, 41)
    stats = _run_staged(cfg, 0, cfg.steps, b_down=True, append_first=1,
                        capacity=F if fire > 0.2 else None)
    assert sum(s["n_evict"] for s in stats) > 0


@pytest.mark.parametrize("two_streams,fused_plan,fused_fetch,S,gate_mode", [
    (True, 1, 1, 1, 0), (True, 0, 1, 1, 0), (True, 1, 0, 1, 0), (False, 1, 1, 1, 0),
    (True, 1, 1, 4, 0), (True, 1, 1, 1, 2), (True, 1, 1, 1, 1)])
def test_append_first_decode_step(two_streams, fused_plan, fused_fetch, S, gate_mode):
    # with two streams the row moves run beside the fetch; all forms must match the oracle
    cfg = W.LifConfig("afd", 1, 512, 4096, 32, 2, S, 14, 0.06, 1.0, 0.8, 0.6, 42)
    act, thr = (B.ACT_FATRELU, 0.05) if gate_mode else (B.ACT_RELU, 0.0)
    gpu, ora = P.make_layer_pair(cfg, 0, append_first=1, gate_mode=gate_mode, activation=act,
                                 act_threshold=thr, b_down=True)
    B.lif_set_tuning(gpu.handle, B.TUNE_FUSED_PLAN, fused_plan)
    B.lif_set_tuning(gpu.handle, B.TUNE_FUSED_FETCH_FFN, fused_fetch)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(S, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = (torch.cuda.Stream(), torch.cuda.Stream()) if two_streams else (None, None)
    torch.cuda.synchronize()
    n_moves = n_reused = 0
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        torch.cuda.synchronize()
        lists = P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
        P.compare_cache_rows(gpu, ora)
        n_moves += len(lists["move_src"])
        n_reused += int((lists["load_slots"] < lists["num_used_before"]).sum())
    st = B.lif_get_stats(gpu.handle)
    assert st.status == B.LIF_OK and st.rows_moved == ora.cache.rows_moved == n_moves
    assert n_reused > 0 and n_moves > 0
    gpu.close()


def test_append_first_with_memory_budget_and_speculative_window():
    cfg = W.LifConfig("afb", 1, 256, 4096, 16, 5, 1, 24, 0.05, 1.0, 0.5, 0.87, 15)
    stats = _run_staged(cfg, 0, cfg.steps, budget_rows=600, capacity=1024, append_first=1)
    assert min(s["k_eff"] for s in stats) < cfg.window_k
    S = 5
    cfg = W.LifConfig("afs", 1, 256, 4096, 16, 3, S, 10, 0.03, 1.0, 0.8, 0.6, 16)
    gpu, ora = P.make_layer_pair(cfg, 0, spec_keep=2, capacity=2048, append_first=1)
    Xs = W.make_inputs(cfg.scaled(n_streams=1, steps=cfg.steps * S), device=DEV)
    X = Xs.reshape(cfg.steps, S, cfg.d_model).contiguous()
    bufs = P.make_bufs(gpu)
    stats = [P.staged_step(gpu, ora, X[t], bufs) for t in range(cfg.steps)]
    assert sum(s["n_evict"] for s in stats) > 0
    gpu.close()


def test_append_first_with_memory_budget_through_the_decode_step():
    cfg = W.LifConfig("afbd", 1, 256, 4096, 16, 5, 1, 24, 0.05, 1.0, 0.5, 0.87, 15)
    gpu, ora = P.make_layer_pair(cfg, 0, budget_rows=600, capacity=1024, append_first=1)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    ks = []
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        torch.cuda.synchronize()
        lists = P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
        P.compare_cache_rows(gpu, ora)
        assert lists["num_used"] <= 600
        ks.append(lists["k_eff"])
    assert min(ks) < cfg.window_k and max(ks) == cfg.window_k, ks
    gpu.close()


def test_append_first_speculative_window_through_the_decode_step():
    S, keep = 5, 2
    cfg = W.LifConfig("afsd", 1, 256, 4096, 16, 3, S, 10, 0.03, 1.0, 0.8, 0.6, 16)
    gpu, ora = P.make_layer_pair(cfg, 0, spec_keep=keep, capacity=2048, append_first=1)
    Xs = W.make_inputs(cfg.scaled(n_streams=1, steps=cfg.steps * S), device=DEV)
    X = Xs.reshape(cfg.steps, S, cfg.d_model).contiguous()
    y = torch.empty(S, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    n_evict = 0
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        g = gpu.lists()
        x_np = X[t].cpu().numpy()
        logits = O.predictor_logits(x_np, ora.A, ora.B, ora.c)
        P.assert_mask_borderline(g["active_idx"], logits, 0.0)
        kt = P.keep_tokens_checked(gpu, g["active_idx"], logits, 0.0)
        _, _, lists, ref_y = O.decode_step(ora.cache, x_np, ora.A, ora.B, ora.c, 0.0, ora.bundles,
                                           ora.bias_up, act=g["active_idx"], keep_token=kt, keep=keep)
        P.compare_lists_and_state(gpu, ora, lists)
        P.compare_cache_rows(gpu, ora)
        P.assert_y_close(y.cpu().numpy().astype(np.float64), ref_y)
        n_evict += len(lists["evict_ids"])
    assert n_evict > 0 and gpu.lists()["step"] == cfg.steps * keep
    gpu.close()


def test_append_first_is_refused_with_the_whole_cache_ffn():
    with pytest.raises(B.LifError) as e:
        B.lif_workspace_bytes(B.make_desc(d_model=256, d_ff=1024, rank=16, window_k=2, capacity=512,
                                          ffn_mode=1, append_first=1))
    assert e.value.code == B.LIF_ERR_INVALID_ARG


@pytest.mark.parametrize("ffn_mode,split,gate_mode", [(0, 1, 0), (0, 0, 0), (1, 1, 0), (1, 0, 0), (0, 1, 1)])
def test_multi_stream_decode_step_split_around_the_fetch(ffn_mode, split, gate_mode):
    # several streams, two CUDA streams: the fetch runs on the second stream, one tensor-core FFN
    # over all rows follows it (the split switch only concerns single-stream layers: splitting the
    # multi-stream FFN around the fetch measured slower)
    cfg = W.LifConfig("msplit", 1, 512, 4096, 32, 2, 3, 10, 0.06, 1.0, 0.8, 0.6, 43)
    act, thr = (B.ACT_FATRELU, 0.05) if gate_mode else (B.ACT_RELU, 0.0)
    gpu, ora = P.make_layer_pair(cfg, 0, ffn_mode=ffn_mode, gate_mode=gate_mode, activation=act,
                                 act_threshold=thr, b_down=True)
    B.lif_set_tuning(gpu.handle, B.TUNE_SPLIT_FFN, split)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(cfg.n_streams, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    n_evict = 0
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        torch.cuda.synchronize()
        x_np = X[t].cpu().numpy()
        if ffn_mode == 0:
            lists = P.check_decode_step(gpu, ora, x_np, y)
        else:
            g = gpu.lists()
            P.assert_mask_borderline(g["active_idx"], ora.scores(x_np), ora.theta)
            lists = ora.cache.window_update(g["active_idx"])
            ora.cache.insert(lists, ora.bundles, ora.bias_up)
            P.compare_lists_and_state(gpu, ora, lists)
            ref_y, flips = P.ffn_reference(ora, np.arange(ora.cache.num_used), x_np)
            P.assert_y_close(y.cpu().numpy().astype(np.float64), ref_y, flips)
        P.compare_cache_rows(gpu, ora)
        n_evict += len(lists["evict_ids"])
    assert n_evict > 0
    gpu.close()


@pytest.mark.parametrize("append_first", [0, 1])
def test_phase_timing_and_snapshot_with_both_cache_orders(append_first):
    cfg = W.CONFIGS["tiny"]
    X = W.make_inputs(cfg, device=DEV)
    gpu, ora = P.make_layer_pair(cfg, 0, append_first=append_first)
    y = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for t in range(6):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
    # event nodes around every kernel of the next three steps (the row moves may run on sf)
    B.lif_timing_enable(gpu.handle, 3)
    for t in range(6, 10):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
    us, n = B.lif_timing_read(gpu.handle)
    assert n == 3 and set(us) == set(B.PHASES)
    assert all(v >= 0.0 for v in us.values()) and us["fetch"] > 0 and us["ffn"] > 0 and us["window"] > 0
    B.lif_timing_enable(gpu.handle, 0)
    # snapshot, run on, wreck, restore, run on again: bitwise the same
    snap = B.lif_snapshot(gpu.handle)
    def run():
        out = []
        for t in range(10, 16):
            B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
            torch.cuda.synchronize()
            out.append((y.cpu().numpy().copy(), gpu.lists()["pointers"].copy()))
        return out
    first = run()
    B.lif_reset(gpu.handle)
    gpu.cache.zero_()
    torch.cuda.synchronize()
    B.lif_restore(gpu.handle, snap)
    again = run()
    for (ya, pa), (yb, pb) in zip(first, again):
        assert np.array_equal(ya.view(np.uint32), yb.view(np.uint32))
        np.testing.assert_array_equal(pa, pb)
    assert gpu.lists()["status"] == B.LIF_OK
    gpu.close()


@pytest.mark.parametrize("gate_mode,append_first", [(0, 0), (0, 1), (2, 1)])
def test_more_neurons_than_the_mask_fed_window_kernel_takes(gate_mode, append_first):
    # d_ff = 40960 > 32768: the decode step uses the list-fed window kernel (the predictor
    # compacts its mask itself); also the widest index range of the gate kernel's mask words
    cfg = W.LifConfig("wide", 1, 256, 40960, 16, 2, 1, 8, 0.02, 1.0, 0.8, 0.6, 51)
    act, thr = (B.ACT_FATRELU, 0.05) if gate_mode else (B.ACT_RELU, 0.0)
    # (a rank-16 predictor makes the active count swing widely from token to token: roomy cache)
    gpu, ora = P.make_layer_pair(cfg, 0, gate_mode=gate_mode, activation=act, act_threshold=thr,
                                 append_first=append_first, capacity=16384)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    n_evict = 0
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        torch.cuda.synchronize()
        assert gpu.lists()["status"] == B.LIF_OK
        lists = P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
        P.compare_cache_rows(gpu, ora)
        n_evict += len(lists["evict_ids"])
    assert n_evict > 0 and gpu.lists()["active_idx"].max() > 32768
    gpu.close()


@pytest.mark.parametrize("d,F,r,k,S", [
    (8, 64, 8, 1, 1),          # the smallest shapes the header allows
    (8, 64, 8, 2, 8),
    (64, 256, 2048, 2, 1),     # the largest predictor rank
    (64, 256, 2048, 2, 8),     # ... with eight streams: 64 KB of stage-1 sums per CTA
    (8192, 264, 8, 2, 2),      # the widest rows, two streams (per-stream FFN: d_model % 16 == 0 but few rows)
])
def test_extreme_shapes(d, F, r, k, S):
    cfg = W.LifConfig("edge", 1, d, F, r, k, S, 8, 0.10, 1.0, 0.8, 0.6, 61)
    stats = _run_staged(cfg, 0, cfg.steps, b_down=True, capacity=F)
    assert max(s["n_active"] for s in stats) > 0
    gpu, ora = P.make_layer_pair(cfg, 0, capacity=F, append_first=1)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(S, d, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        torch.cuda.synchronize()
        P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
        P.compare_cache_rows(gpu, ora)
    gpu.close()


@pytest.mark.parametrize("gate_mode,act", [(1, B.ACT_RELU_SQUARED), (0, B.ACT_RELU_SQUARED), (0, B.ACT_RELU)])
def test_multi_stream_ffn_with_tiny_activations(gate_mode, act):
    # d_model = 16 and squared ReLU give activations around 1e-5 and below: the tensor-core FFN
    # splits them into fp16 parts and must not lose them to fp16's narrow exponent range
    cfg = W.LifConfig("tinyact", 1, 16, 2000, 40, 6, 8, 10, 0.01, 1.0, 0.8, 0.6, 551)
    gpu, ora = P.make_layer_pair(cfg, 0, gate_mode=gate_mode, activation=act, capacity=2000)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(8, 16, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
    gpu.close()


@pytest.mark.parametrize("early,two_streams,append_first,S,gate_mode", [
    (1, True, 1, 3, 0), (0, True, 1, 3, 0), (1, True, 0, 3, 0), (1, False, 1, 3, 0), (1, False, 0, 8, 0),
    (1, True, 1, 1, 1), (0, True, 1, 1, 1), (1, True, 0, 1, 1), (1, True, 1, 4, 1)])
def test_fetch_as_a_kernel_of_its_own_early_or_after_the_lists(early, two_streams, append_first, S,
                                                              gate_mode):
    # several input streams, or three-vector bundles: the fetch is not fused with the FFN; by
    # default it starts from the predictor's masks while the window kernel runs, with the knob
    # off it waits for the lists.  A predictor call with another input between the steps leaves
    # masks that are not the step's.
    cfg = W.LifConfig("efetch", 1, 512, 4096, 32, 2, S, 12, 0.06, 1.0, 0.8, 0.6, 47)
    act, thr = (B.ACT_FATRELU, 0.05) if gate_mode else (B.ACT_RELU, 0.0)
    gpu, ora = P.make_layer_pair(cfg, 0, gate_mode=gate_mode, activation=act, act_threshold=thr,
                                 b_down=True, append_first=append_first)
    B.lif_set_tuning(gpu.handle, B.TUNE_EARLY_FETCH, early)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(S, cfg.d_model, dtype=torch.float32, device=DEV)
    idx = torch.empty(cfg.d_ff, dtype=torch.int32, device=DEV)
    n = torch.zeros(1, dtype=torch.int32, device=DEV)
    sc, sf = (torch.cuda.Stream(), torch.cuda.Stream()) if two_streams else (None, None)
    torch.cuda.synchronize()
    n_load = n_evict = 0
    for t in range(cfg.steps):
        if t % 3 == 1:
            B.lif_predict(gpu.handle, X[(t + 4) % cfg.steps], None, idx, n, sc)
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        lists = P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
        P.compare_cache_rows(gpu, ora)
        n_load += len(lists["load_ids"])
        n_evict += len(lists["evict_ids"])
    assert n_load > 148 and n_evict > 0          # more rows than CTAs in some step, and row reuse
    gpu.close()
