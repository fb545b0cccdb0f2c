"""Full-size parity of the named configurations, run the way the benchmark runs them: the whole
stack, one CUDA graph per token.  The oracle follows a sample of layers token by token (teacher
forced from the GPU's active lists); every other layer is checked through properties that hold
at any size (status, traffic accounting, cache structure, cached rows bit-identical to the
host store)."""
import numpy as np
import psutil
import pytest
import torch

from paper_2312_11514_b200 import binding as B
from paper_2312_11514_b200 import runtime as R
from paper_2312_11514_b200 import workloads as W

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run_config(name, n_tokens, sample_layers, oracle_tokens=None, gate_mode=0, activation=0, thr=0.0,
                append_first=0):
    cfg = W.CONFIGS[name]
    n_vec = 3 if gate_mode == B.GATE_BUNDLED else 2
    bundle_bytes = n_vec * cfg.d_model * 2
    store_gib = cfg.n_layers * cfg.d_ff * bundle_bytes / 2**30
    if psutil.virtual_memory().available / 2**30 < store_gib * 1.3 + 8:
        pytest.skip(f"host memory too small for the {store_gib:.0f} GiB bundle store")
    n_tokens = min(n_tokens, cfg.steps)
    oracle_tokens = n_tokens if oracle_tokens is None else min(oracle_tokens, n_tokens)
    L, S, d, F = cfg.n_layers, cfg.n_streams, cfg.d_model, cfg.d_ff
    layers, oras = [], {}
    for l in range(L):
        store = R.pinned_store(F, d, n_vec)
        w = W.make_layer(cfg, l, device=DEV, bundles_out=store, gate_mode=gate_mode, act_threshold=thr)
        cap = W.window_capacity(cfg, w["p"])
        layers.append(R.Layer(d_model=d, d_ff=F, rank=cfg.rank, window_k=cfg.window_k, capacity=cap,
                              host_bundles=store, pred_A=w["A"], pred_B=w["B"], pred_c=w["c"],
                              bias_up=w["bias_up"], n_streams=S, gate_mode=gate_mode, gate=w.get("gate"),
                              activation=activation, activation_threshold=thr,
                              append_first=append_first, device=DEV))
        if l in sample_layers:
            oras[l] = P.OracleLayer(w, d, F, cap, cfg.window_k, activation=activation,
                                    act_threshold=thr, gate_mode=gate_mode, append_first=append_first)
        del w
    X = W.make_inputs(cfg, device=DEV)
    dev_x = torch.empty(S, d, dtype=torch.float16, device=DEV)
    Y = torch.zeros(L, S, d, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    graph = B.lif_graph_capture([l.handle for l in layers], dev_x, Y, sc, sf)
    n_loaded = 0
    for t in range(n_tokens):
        with torch.cuda.stream(sc):
            dev_x.copy_(X[t])
        B.lif_graph_launch(graph, sc)
        torch.cuda.synchronize()
        if t >= oracle_tokens:
            continue
        x_np = X[t].cpu().numpy()
        y_np = Y.cpu().numpy().astype(np.float64)
        for l, ora in oras.items():
            lists = P.check_decode_step(layers[l], ora, x_np, y_np[l])
            n_loaded += len(lists["load_ids"])
    # every layer: properties that hold at any size
    for l, lay in enumerate(layers):
        st = B.lif_get_stats(lay.handle)
        g = lay.lists()
        assert st.status == B.LIF_OK, (l, st.status)
        n = g["num_used"]
        assert g["step"] == n_tokens and 0 < n <= lay.capacity
        assert st.bytes_fetched % bundle_bytes == 0 and st.bytes_fetched >= n * bundle_bytes
        ptr = g["pointers"][:n]
        assert len(np.unique(ptr)) == n and ptr.min() >= 0
        assert (g["slot_of"][ptr] == np.arange(n)).all() and (g["slot_of"] >= 0).sum() == n
        assert (g["last_active"][ptr] > n_tokens - 1 - cfg.window_k).all()      # inside the window
        assert (g["last_active"][g["active_idx"]] == n_tokens - 1).all()
        rows = lay.cache[:n].cpu()
        want = lay.keep["host_bundles"][torch.from_numpy(ptr.astype(np.int64))]
        assert torch.equal(rows.view(torch.int16), want.view(torch.int16)), f"layer {l} cache rows"
        bias_want = lay.keep["bias_up"].cpu()[torch.from_numpy(ptr.astype(np.int64))]
        assert torch.equal(torch.from_numpy(g["bias"][:n]).view(torch.int16), bias_want.view(torch.int16))
    for l, ora in oras.items():
        if oracle_tokens == n_tokens:
            P.compare_cache_rows(layers[l], ora)
    assert n_loaded > 0
    B.lif_graph_destroy(graph)
    for lay in layers:
        lay.close()


def test_opt6p7b_full_stack_all_tokens():
    _run_config("opt6p7b", 128, sample_layers=(0, 15, 31))


def test_opt6p7b_full_stack_new_neurons_stacked_first():
    # the benchmark's default order of the cache operations: bundles go straight into freed rows
    _run_config("opt6p7b", 48, sample_layers=(0, 15, 31), append_first=1)


def test_falcon7b_full_stack():
    _run_config("falcon7b", 48, sample_layers=(3, 30), oracle_tokens=40)


def test_phi2_full_stack():
    _run_config("phi2", 64, sample_layers=(0, 17), oracle_tokens=48)


def test_batched8_full_stack_eight_streams():
    _run_config("batched8", 8, sample_layers=(1, 46), oracle_tokens=6, append_first=1)


@pytest.mark.parametrize("gate_mode", [B.GATE_BUNDLED, B.GATE_RESIDENT])
def test_llama2_7b_gated_full_stack(gate_mode):
    # Appendix C, Llama 2: gated FFN with FATReLU, window of 2; the gate row either travels in
    # the bundle (low-rank predictor) or stays resident and is the predictor
    _run_config("llama2_7b", 32, sample_layers=(0, 20), oracle_tokens=24, gate_mode=gate_mode,
                activation=B.ACT_FATRELU, thr=0.05)
