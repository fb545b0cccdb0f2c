"""Seeded random configurations through the staged entry points and through lif_decode_step,
against the oracle: shapes, window sizes, stream counts, firing rates, activations, gate modes,
both orders of the cache operations and the launch-shape switches, drawn together."""
import numpy as np
import pytest
import torch

from paper_2312_11514_b200 import binding as B
from paper_2312_11514_b200 import workloads as W

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _draw(rng):
    d = int(rng.choice([8, 16, 64, 136, 256, 520, 1024, 2048]))
    F = int(rng.integers(8, 700)) * 8
    r = int(rng.choice([8, 16, 40, 128, 256]))
    k = int(rng.integers(1, 7))
    S = int(rng.choice([1, 1, 1, 2, 3, 5, 8]))
    fire = float(rng.choice([0.01, 0.02, 0.05, 0.2, 0.5]))
    gate_mode = int(rng.choice([0, 0, 1, 2]))
    act = int(rng.choice([0, 1, 2]))
    append_first = int(rng.integers(0, 2))
    ffn_mode = 0 if append_first else int(rng.integers(0, 2))
    cfg = W.LifConfig("random", 1, d, F, r, k, S, 6, fire, 1.0, 0.8, 0.6, int(rng.integers(0, 1000)))
    kw = dict(gate_mode=gate_mode, activation=act, act_threshold=0.05 if act == 2 else 0.0,
              append_first=append_first, ffn_mode=ffn_mode, capacity=F, b_down=bool(rng.integers(0, 2)))
    return cfg, kw


@pytest.mark.parametrize("seed", [0, 1, 2, 3, 4, 5])
def test_random_configurations(seed):
    rng = np.random.default_rng(1000 + seed)
    for _ in range(12):
        cfg, kw = _draw(rng)
        staged = bool(rng.integers(0, 2))
        tune = [(B.TUNE_FUSED_PLAN, int(rng.integers(0, 2))), (B.TUNE_FUSED_FETCH_FFN, int(rng.integers(0, 2))),
                (B.TUNE_DEPENDENT_LAUNCH, int(rng.integers(0, 2)))]
        two_streams = bool(rng.integers(0, 2))
        where = f"{cfg} {kw} staged={staged} tune={tune} two_streams={two_streams}"
        gpu, ora = P.make_layer_pair(cfg, 0, **kw)
        X = W.make_inputs(cfg, device=DEV)
        whole = kw["ffn_mode"] == 1
        try:
            if staged:
                bufs = P.make_bufs(gpu)
                for t in range(cfg.steps):
                    P.staged_step(gpu, ora, X[t], bufs, whole_cache=whole)
            else:
                for key, value in tune:
                    B.lif_set_tuning(gpu.handle, key, value)
                y = torch.empty(cfg.n_streams, cfg.d_model, dtype=torch.float32, device=DEV)
                sc, sf = (torch.cuda.Stream(), torch.cuda.Stream()) if two_streams else (None, None)
                torch.cuda.synchronize()
                for t in range(cfg.steps):
                    B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
                    x_np = X[t].cpu().numpy()
                    if not whole:
                        P.check_decode_step(gpu, ora, x_np, y)
                    else:
                        g = gpu.lists()
                        assert g["status"] == B.LIF_OK
                        scores = ora.scores(x_np)
                        P.assert_mask_borderline(g["active_idx"], scores, ora.theta)
                        lists = ora.cache.window_update(g["active_idx"])
                        ora.cache.insert(lists, ora.bundles, ora.bias_up)
                        P.compare_lists_and_state(gpu, ora, lists)
                        slots = np.arange(ora.cache.num_used)
                        gate_pre = scores[:, ora.cache.pointers[slots]] if kw["gate_mode"] == 2 else None
                        ref_y, flips = P.ffn_reference(ora, slots, x_np, gate_pre)
                        P.assert_y_close(y.cpu().numpy().astype(np.float64), ref_y, flips)
                    P.compare_cache_rows(gpu, ora)
        except AssertionError as e:
            raise AssertionError(f"{where}: {e}") from e
        finally:
            gpu.close()
