"""GPU parity of the gated FFN (Appendix C, Llama 2): three-vector bundles behind the low-rank
predictor, and the resident gate projection as the predictor, through the staged entry points
and through lif_decode_step, single- and multi-stream."""
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


def _staged(cfg, **kw):
    gpu, ora = P.make_layer_pair(cfg, 0, **kw)
    X = W.make_inputs(cfg, device=DEV)
    bufs = P.make_bufs(gpu)
    stats = [P.staged_step(gpu, ora, X[t], bufs, whole_cache=kw.get("ffn_mode", 0) == 1)
             for t in range(cfg.steps)]
    st = B.lif_get_stats(gpu.handle)
    n_vec = 3 if kw.get("gate_mode") == B.GATE_BUNDLED else 2
    assert st.status == B.LIF_OK
    assert st.bytes_fetched == ora.cache.bytes_fetched == \
        sum(s["n_load"] for s in stats) * n_vec * cfg.d_model * 2
    gpu.close()
    return stats


@pytest.mark.parametrize("gate_mode", [B.GATE_BUNDLED, B.GATE_RESIDENT])
@pytest.mark.parametrize("d,F,r,k,S,act,thr", [
    (256, 1024, 16, 3, 1, B.ACT_FATRELU, 0.05),
    (264, 1000, 24, 2, 1, B.ACT_RELU, 0.0),           # ragged: nothing a multiple of the tiles
    (4096, 1408, 32, 2, 1, B.ACT_FATRELU, 0.1),       # Llama 2 7B row length
    (512, 4096, 40, 2, 3, B.ACT_FATRELU, 0.05),       # three streams
    (256, 1536, 16, 2, 8, B.ACT_RELU_SQUARED, 0.0),   # eight streams
    (8192, 520, 16, 2, 1, B.ACT_FATRELU, 0.1),        # widest rows, last tile of 8 neurons
    (2048, 2048, 16, 2, 8, B.ACT_FATRELU, 0.05),      # eight streams, tensor-core FFN
])
def test_gated_staged(gate_mode, d, F, r, k, S, act, thr):
    cfg = W.LifConfig("gated", 1, d, F, r, k, S, 8, 0.08, 1.0, 0.8, 0.6, 21)
    stats = _staged(cfg, gate_mode=gate_mode, activation=act, act_threshold=thr, b_down=True)
    assert sum(s["n_evict"] for s in stats) > 0 and min(s["n_active"] for s in stats) > 0


@pytest.mark.parametrize("gate_mode", [B.GATE_BUNDLED, B.GATE_RESIDENT])
def test_gated_whole_cache_mode(gate_mode):
    cfg = W.LifConfig("gatedw", 1, 512, 2048, 16, 3, 1, 6, 0.10, 1.0, 0.8, 0.6, 22)
    _staged(cfg, gate_mode=gate_mode, activation=B.ACT_FATRELU, act_threshold=0.05, ffn_mode=1)


@pytest.mark.parametrize("gate_mode,S,two_streams,fused", [
    (B.GATE_BUNDLED, 1, True, 1), (B.GATE_BUNDLED, 1, False, 0), (B.GATE_BUNDLED, 4, True, 1),
    (B.GATE_RESIDENT, 1, True, 1), (B.GATE_RESIDENT, 1, False, 0), (B.GATE_RESIDENT, 4, True, 1)])
def test_gated_decode_step(gate_mode, S, two_streams, fused):
    cfg = W.LifConfig("gatedd", 1, 512, 4096, 32, 2, S, 10, 0.06, 1.0, 0.8, 0.6, 23)
    thr = 0.05
    gpu, ora = P.make_layer_pair(cfg, 0, gate_mode=gate_mode, activation=B.ACT_FATRELU,
                                 act_threshold=thr, b_down=True)
    B.lif_set_tuning(gpu.handle, B.TUNE_FUSED_PLAN, fused)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(S, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = (torch.cuda.Stream(), torch.cuda.Stream()) if two_streams else (None, None)
    torch.cuda.synchronize()
    n_evict = 0
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        lists = P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
        P.compare_cache_rows(gpu, ora)
        n_evict += len(lists["evict_ids"])
    assert n_evict > 0
    gpu.close()


def test_resident_gate_output_is_the_dense_gated_ffn():
    # the resident gate finds exactly the neurons with a non-zero activation, so every step's
    # output is the dense gated FFN over all d_ff neurons (computed here from the full weights)
    cfg = W.LifConfig("gatedx", 1, 256, 2048, 16, 2, 1, 6, 0.08, 1.0, 0.8, 0.6, 24)
    thr = 0.05
    gpu, ora = P.make_layer_pair(cfg, 0, gate_mode=B.GATE_RESIDENT, activation=B.ACT_FATRELU,
                                 act_threshold=thr)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
    Wg, bg = ora.gate.astype(np.float64), ora.bias_up.astype(np.float64)
    Wu = ora.bundles[:, :cfg.d_model].astype(np.float64)
    Wd = ora.bundles[:, cfg.d_model:].astype(np.float64)
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y)
        x = X[t].cpu().numpy().astype(np.float64)
        g = x @ Wg.T + bg
        u = x @ Wu.T
        dense = (np.where(g > thr, g, 0.0) * u) @ Wd
        flips = [(0, (-1.0 if g[0, i] > thr else 1.0) * g[0, i] * u[0, i] * Wd[i])
                 for i in np.nonzero(np.abs(g[0] - thr) < P.ACT_BORDER)[0]]   # decisions within rounding
        P.assert_y_close(y.cpu().numpy().astype(np.float64), dense, flips)
        assert gpu.lists()["status"] == B.LIF_OK
    gpu.close()


def test_gate_mode_argument_checks():
    cfg = W.LifConfig("gatedc", 1, 256, 1024, 16, 2, 2, 4, 0.08, 1.0, 0.8, 0.6, 25)
    store = R.pinned_store(cfg.d_ff, cfg.d_model)
    w = W.make_layer(cfg, 0, device=DEV, bundles_out=store, gate_mode=B.GATE_RESIDENT)
    with pytest.raises(B.LifError) as e:          # resident gate without the gate matrix
        R.Layer(d_model=cfg.d_model, d_ff=cfg.d_ff, rank=cfg.rank, window_k=2, capacity=512,
                host_bundles=store, bias_up=w["bias_up"], n_streams=2, gate_mode=B.GATE_RESIDENT)
    assert e.value.code == B.LIF_ERR_INVALID_ARG
    with pytest.raises(B.LifError) as e:          # resident gate with a speculative window
        B.lif_workspace_bytes(B.make_desc(d_model=256, d_ff=1024, rank=16, window_k=2, capacity=512,
                                          n_streams=2, spec_keep=1, gate_mode=B.GATE_RESIDENT))
    assert e.value.code == B.LIF_ERR_INVALID_ARG
    with pytest.raises(B.LifError):
        B.lif_workspace_bytes(B.make_desc(d_model=256, d_ff=1024, rank=16, window_k=2, capacity=512,
                                          gate_mode=3))
