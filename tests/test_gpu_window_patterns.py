"""Chosen active sets through lif_decode_step.  A predictor with a zero first factor makes the
scores equal to the per-neuron offsets, which the test rewrites before every token, so the
window kernels see exactly the sets listed here: empty sets, complete turnover, everything at
once (more rows and denser mask words than the register-resident window kernel takes, so it
hands over inside the launch), single neurons at both ends of the id range, complements.
Lists, slot maps and state must match the oracle bit for bit, the output within tolerance."""
import numpy as np
import pytest
import torch

from paper_2312_11514_b200 import binding as B
from paper_2312_11514_b200 import runtime as R
from paper_2312_11514_b200 import workloads as W

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _patterns(F, rng):
    every = np.arange(F)
    rand_a = np.nonzero(rng.random(F) < 0.3)[0]
    rand_b = np.nonzero(rng.random(F) < 0.3)[0]
    dense_words = every[(every // 32) % 5 == 0]                 # whole 32-neuron mask words
    return [
        ("empty", every[:0]), ("block", every[:700]), ("same block", every[:700]),
        ("disjoint block", every[700:1500]), ("empty", every[:0]), ("empty again", every[:0]),
        ("everything", every), ("every 7th", every[::7]), ("last id", every[-1:]),
        ("first id", every[:1]), ("random", rand_a), ("random, redrawn", rand_b),
        ("complement", np.setdiff1d(every, rand_b)), ("whole mask words", dense_words),
        ("ragged last word", every[F - F % 32 - 40:]), ("empty", every[:0]),
    ]


@pytest.mark.parametrize("fused_plan,append_first,k", [(1, 0, 2), (0, 0, 2), (1, 1, 2), (0, 1, 3), (1, 1, 1)])
def test_chosen_active_sets(fused_plan, append_first, k):
    d, F, r = 64, 5000, 8                                       # 5000 = 156 mask words + 8 ids
    cfg = W.LifConfig("patterns", 1, d, F, r, k, 1, 16, 0.05, 1.0, 0.8, 0.6, 57)
    store = R.pinned_store(F, d)
    w = W.make_layer(cfg, 0, device=DEV, bundles_out=store)
    w["A"] = torch.zeros_like(w["A"])                           # scores = offsets c, exactly
    w["c"] = torch.full((F,), -1.0, dtype=torch.float32, device=DEV)
    gpu = R.Layer(d_model=d, d_ff=F, rank=r, window_k=k, capacity=F, host_bundles=store,
                  pred_A=w["A"], pred_B=w["B"], pred_c=w["c"], bias_up=w["bias_up"],
                  append_first=append_first, device=DEV)
    ora = P.OracleLayer(w, d, F, F, k, append_first=append_first)
    B.lif_set_tuning(gpu.handle, B.TUNE_FUSED_PLAN, fused_plan)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(1, d, dtype=torch.float32, device=DEV)
    history = []
    for t, (name, ids) in enumerate(_patterns(F, np.random.default_rng(5))):
        c = np.full(F, -1.0, dtype=np.float32)
        c[ids] = 1.0
        w["c"].copy_(torch.from_numpy(c))
        ora.c[:] = c
        torch.cuda.synchronize()
        B.lif_decode_step(gpu.handle, X[t], y)
        torch.cuda.synchronize()
        lists = P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
        np.testing.assert_array_equal(gpu.lists()["active_idx"], ids, err_msg=name)
        P.compare_cache_rows(gpu, ora)
        history.append(set(ids.tolist()))
        assert ora.cache.cached_ids() == set().union(*history[-k:]), name
        assert lists["num_used"] == len(ora.cache.cached_ids())
    gpu.close()
