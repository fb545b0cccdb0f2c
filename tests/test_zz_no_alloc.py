"""lif_sparse_ffn_static — the sparse FFN for callers that cannot allocate device memory
(plugin code under a foreign allocator, processes whose memory is already handed out, paths
that must not trigger the implicit synchronisation of cudaMalloc/cudaFree).  It keeps its
partial sums in a fixed array inside the library, so this file checks two things: that it
computes what lif_sparse_ffn computes, and that a second call is not polluted by what the
first one left in that shared array.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_2312_11514_b200 import binding as B
from paper_2312_11514_b200 import workloads as W

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_static_scratch_ffn_matches_workspace_ffn_on_two_calls_in_a_row():
    cfg = W.LifConfig("noalloc", 1, 1032, 4096, 32, 3, 1, 4, 0.10, 1.0, 0.8, 0.6, 21)
    gpu, ora = P.make_layer_pair(cfg, 0, b_down=True)
    X = W.make_inputs(cfg, device=DEV)
    # fill the cache through the normal path so both entry points read the same rows
    y_tmp = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
    for t in range(3):
        B.lif_decode_step(gpu.handle, X[t], y_tmp)
    g = gpu.lists()
    assert g["status"] == B.LIF_OK and g["num_used"] > 300
    bias = gpu._view("bias", gpu.capacity, torch.float16)
    b_down = gpu.keep["bias_down"]
    n_all = torch.tensor([g["num_used"]], dtype=torch.int32, device=DEV)
    # call 1: every cached row; call 2: a short explicit slot list (far fewer CTAs take part,
    # so most of the array still holds call 1's partial sums)
    few = torch.tensor([7, 3, 250, 11, 42], dtype=torch.int32, device=DEV)
    n_few = torch.tensor([5], dtype=torch.int32, device=DEV)
    for slots, n in ((None, n_all), (few, n_few)):
        want = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
        got = torch.full((cfg.d_model,), float("nan"), dtype=torch.float32, device=DEV)
        B.lif_sparse_ffn(gpu.handle, X[3], slots, n, want)
        B.lif_sparse_ffn_static(gpu.cache, bias, X[3], slots, n, b_down, got, cfg.d_model)
        torch.cuda.synchronize()
        P.assert_y_close(got.cpu().numpy().astype(np.float64)[None, :],
                         want.cpu().numpy().astype(np.float64))
        assert torch.isfinite(got).all() and got.abs().max() > 0
    # zero rows: only the down bias is left, whatever the array holds
    got = torch.empty(cfg.d_model, dtype=torch.float32, device=DEV)
    B.lif_sparse_ffn_static(gpu.cache, bias, X[3], None, torch.zeros(1, dtype=torch.int32, device=DEV),
                            b_down, got, cfg.d_model)
    torch.cuda.synchronize()
    assert torch.equal(got, b_down.float())
    gpu.close()


def test_static_scratch_ffn_rejects_sizes_beyond_its_array():
    x = torch.zeros(16384, dtype=torch.float16, device=DEV)
    y = torch.zeros(16384, dtype=torch.float32, device=DEV)
    n = torch.zeros(1, dtype=torch.int32, device=DEV)
    for d_bad in (8200, 16384, 12, 0):
        with pytest.raises(B.LifError) as e:
            B.lif_sparse_ffn_static(x, x, x, None, n, None, y, d_bad)
        assert e.value.code == B.LIF_ERR_INVALID_ARG
    with pytest.raises(B.LifError) as e:
        B.lif_sparse_ffn_static(x, x, x[1:], None, n, None, y, 256)
    assert e.value.code == B.LIF_ERR_ALIGNMENT
