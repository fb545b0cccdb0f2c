"""The synthetic generator: shapes, determinism and the calibrated rates of the tiny config."""
import numpy as np
import torch

from oracle import lif_oracle as O
from paper_2312_11514_b200 import workloads as W


def test_config_table_matches_named_shapes():
    c = W.CONFIGS
    assert (c["tiny"].d_model, c["tiny"].d_ff, c["tiny"].rank, c["tiny"].steps) == (256, 1024, 16, 32)
    assert (c["opt6p7b"].n_layers, c["opt6p7b"].d_model, c["opt6p7b"].d_ff, c["opt6p7b"].rank) == (32, 4096, 16384, 128)
    assert c["opt6p7b"].bundle_bytes == 16384                        # 16 KB per neuron
    assert (c["falcon7b"].d_model, c["falcon7b"].d_ff) == (4544, 18176)
    assert (c["phi2"].d_model, c["phi2"].d_ff, c["phi2"].window_k) == (2560, 10240, 4)
    assert (c["batched8"].n_streams, c["batched8"].n_layers, c["batched8"].d_model) == (8, 48, 7168)
    store = c["batched8"].n_layers * c["batched8"].d_ff * c["batched8"].bundle_bytes
    assert abs(store / 2**30 - 36.75) < 0.01


def test_tiny_layer_is_deterministic_and_calibrated():
    cfg = W.CONFIGS["tiny"]
    a, b = W.make_layer(cfg, 0), W.make_layer(cfg, 0)
    for key in ("bundles", "bias_up", "A", "B", "c"):
        assert torch.equal(a[key], b[key])
    assert not torch.equal(a["bundles"], W.make_layer(cfg, 1)["bundles"])
    assert a["bundles"].shape == (1024, 512) and a["bundles"].dtype == torch.float16
    assert abs(a["p"].mean().item() - 0.05) < 1e-6
    assert abs(a["bundles"].float().std().item() - 0.02) < 1e-3
    # N(0, I) inputs: predicted density and true firing rate both ~ mean(p)
    g = torch.Generator().manual_seed(123)
    X = torch.randn(400, cfg.d_model, generator=g, dtype=torch.float64).numpy()
    logits = O.predictor_logits(X, a["A"].numpy(), a["B"].numpy(), a["c"].numpy())
    assert abs((logits > 0).mean() - 0.05) < 0.01
    pre = X @ a["bundles"][:, :cfg.d_model].double().numpy().T + a["bias_up"].double().numpy()
    assert abs((pre > 0).mean() - 0.05) < 0.01


def test_inputs_ar1_and_capacity():
    cfg = W.CONFIGS["tiny"]
    X = W.make_inputs(cfg)
    assert X.shape == (32, 1, 256) and X.dtype == torch.float16
    assert torch.equal(X, W.make_inputs(cfg))
    x = X[:, 0].double().numpy()
    corr = np.mean([np.corrcoef(x[t], x[t + 1])[0, 1] for t in range(31)])
    assert abs(corr - 0.8) < 0.08
    assert abs(x.std() - 1.0) < 0.1
    lay = W.make_layer(cfg, 0)
    cap = W.window_capacity(cfg, lay["p"])
    assert cap % 64 == 0 and 128 < cap <= 1024
    # the capacity recipe covers the real window union of this seed
    cache = O.NeuronCache(cfg.d_model, cfg.d_ff, cap, cfg.window_k)
    for t in range(cfg.steps):
        act = O.active_set(O.predictor_logits(X[t].numpy(), lay["A"].numpy(), lay["B"].numpy(),
                                              lay["c"].numpy()), 0.0)
        cache.window_update(act)
    assert cache.num_used <= cap


def test_gated_layers_shapes_and_gate_firing_rate():
    cfg = W.CONFIGS["tiny"]
    d, F, thr = cfg.d_model, cfg.d_ff, 0.05
    plain = W.make_layer(cfg, 0)
    bun = W.make_layer(cfg, 0, gate_mode=W.GATE_BUNDLED, act_threshold=thr)
    res = W.make_layer(cfg, 0, gate_mode=W.GATE_RESIDENT, act_threshold=thr)
    assert bun["bundles"].shape == (F, 3 * d) and "gate" not in bun
    assert res["bundles"].shape == (F, 2 * d) and res["gate"].shape == (F, d)
    # the same draws: the resident gate is the first vector of the three-vector bundle
    assert torch.equal(res["gate"], bun["bundles"][:, :d])
    assert torch.equal(res["bundles"], bun["bundles"][:, d:])
    assert torch.equal(res["bias_up"], bun["bias_up"])
    assert plain["bundles"].shape == (F, 2 * d)
    assert W.CONFIGS["llama2_7b"].d_ff == 11008 and W.CONFIGS["llama2_7b"].window_k == 2
    # N(0, I) inputs: the gate value passes the threshold at the configured mean rate, and the
    # resident gate as predictor finds exactly those neurons
    g = torch.Generator().manual_seed(7)
    X = torch.randn(400, d, generator=g, dtype=torch.float64).numpy()
    scores = O.gate_scores(X, res["gate"].numpy(), res["bias_up"].numpy())
    assert abs((scores > thr).mean() - cfg.mean_fire) < 0.01
    pre = X @ bun["bundles"][:, :d].double().numpy().T + bun["bias_up"].double().numpy()
    np.testing.assert_allclose(pre, scores, rtol=1e-12, atol=1e-12)
