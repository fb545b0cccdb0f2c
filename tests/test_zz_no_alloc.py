"""lif_sparse_ffn_static — the sparse FFN for callers that cannot allocate device memory
(plugin code under a foreign allocator, processes whose memory is already handed out, paths
that must not trigger the implicit synchronisation of cudaMalloc/cudaFree).  It keeps its
partial sums in a fixed array inside the library, so this file checks three things: that it
computes what lif_sparse_ffn computes and what the CPU oracle computes from the same rows,
that a second call is not polluted by what the first one left in that shared array, and that
what only its kernels can see (a row outside the matrix) reaches the caller through
lif_sparse_ffn_static_status.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import lif_oracle as O
from paper_2312_11514_b200 import binding as B
from paper_2312_11514_b200 import workloads as W

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _filled_layer():
    cfg = W.LifConfig("noalloc", 1, 1032, 4096, 32, 3, 1, 4, 0.10, 1.0, 0.8, 0.6, 21)
    gpu, ora = P.make_layer_pair(cfg, 0, b_down=True)
    X = W.make_inputs(cfg, device=DEV)
    # fill the cache through the normal path so both entry points read the same rows
    y_tmp = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
    for t in range(3):
        B.lif_decode_step(gpu.handle, X[t], y_tmp)
    g = gpu.lists()
    assert g["status"] == B.LIF_OK and g["num_used"] > 300
    return cfg, gpu, X, g


def _oracle_y(gpu, x, rows):
    """The oracle's sparse FFN (float64) over the given rows of the GPU's own cache."""
    matrix = gpu.cache.cpu().numpy()
    bias = gpu._view("bias", gpu.capacity, torch.float16).cpu().numpy()
    b_down = gpu.keep["bias_down"].cpu().numpy()
    return O.sparse_ffn(matrix, bias, np.asarray(rows, dtype=np.int64),
                        x.cpu().numpy().reshape(1, -1), b_down)


def test_static_scratch_ffn_matches_workspace_ffn_on_two_calls_in_a_row():
    cfg, gpu, X, g = _filled_layer()
    B.lif_sparse_ffn_static_status()                       # start from a clear status word
    bias = gpu._view("bias", gpu.capacity, torch.float16)
    b_down = gpu.keep["bias_down"]
    n_all = torch.tensor([g["num_used"]], dtype=torch.int32, device=DEV)
    # call 1: every cached row; call 2: a short explicit slot list (far fewer CTAs take part,
    # so most of the array still holds call 1's partial sums); the last cached row is in it
    few_rows = [7, 3, 250, 11, g["num_used"] - 1]
    few = torch.tensor(few_rows, dtype=torch.int32, device=DEV)
    n_few = torch.tensor([5], dtype=torch.int32, device=DEV)
    for slots, n, rows in ((None, n_all, range(g["num_used"])), (few, n_few, few_rows)):
        want = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
        got = torch.full((cfg.d_model,), float("nan"), dtype=torch.float32, device=DEV)
        B.lif_sparse_ffn(gpu.handle, X[3], slots, n, want)
        B.lif_sparse_ffn_static(gpu.cache, gpu.capacity, bias, X[3], slots, n, b_down, got, cfg.d_model)
        torch.cuda.synchronize()
        got64 = got.cpu().numpy().astype(np.float64)[None, :]
        P.assert_y_close(got64, want.cpu().numpy().astype(np.float64))
        P.assert_y_close(got64, _oracle_y(gpu, X[3], rows))
        assert torch.isfinite(got).all() and got.abs().max() > 0
    # zero rows: only the down bias is left, whatever the array holds
    got = torch.empty(cfg.d_model, dtype=torch.float32, device=DEV)
    B.lif_sparse_ffn_static(gpu.cache, gpu.capacity, bias, X[3], None,
                            torch.zeros(1, dtype=torch.int32, device=DEV), b_down, got, cfg.d_model)
    torch.cuda.synchronize()
    assert torch.equal(got, b_down.float())
    assert B.lif_sparse_ffn_static_status() == B.LIF_OK
    gpu.close()


def test_static_scratch_ffn_refuses_rows_outside_the_matrix_and_says_so():
    # Rows outside [0, n_rows) and a count beyond n_rows are never used as addresses: the call
    # computes the FFN over the valid entries and the status word reports the bad input until
    # it is read.
    cfg, gpu, X, g = _filled_layer()
    B.lif_sparse_ffn_static_status()
    bias = gpu._view("bias", gpu.capacity, torch.float16)
    b_down = gpu.keep["bias_down"]
    n_rows = g["num_used"]                    # tell the call that the matrix ends here
    rows = [5, n_rows, 17, -1, n_rows - 1, 2 ** 30]
    valid = [r for r in rows if 0 <= r < n_rows]
    slots = torch.tensor(rows, dtype=torch.int32, device=DEV)
    n = torch.tensor([len(rows)], dtype=torch.int32, device=DEV)
    got = torch.full((cfg.d_model,), float("nan"), dtype=torch.float32, device=DEV)
    B.lif_sparse_ffn_static(gpu.cache, n_rows, bias, X[3], slots, n, b_down, got, cfg.d_model)
    assert B.lif_sparse_ffn_static_status(clear=False) == B.LIF_ERR_INVALID_ARG
    assert B.lif_sparse_ffn_static_status() == B.LIF_ERR_INVALID_ARG      # sticky until cleared
    assert B.lif_sparse_ffn_static_status() == B.LIF_OK
    P.assert_y_close(got.cpu().numpy().astype(np.float64)[None, :], _oracle_y(gpu, X[3], valid))
    # a count beyond the matrix is clamped to it
    too_many = torch.tensor([n_rows + 1000], dtype=torch.int32, device=DEV)
    B.lif_sparse_ffn_static(gpu.cache, n_rows, bias, X[3], None, too_many, b_down, got, cfg.d_model)
    assert B.lif_sparse_ffn_static_status() == B.LIF_ERR_INVALID_ARG
    P.assert_y_close(got.cpu().numpy().astype(np.float64)[None, :], _oracle_y(gpu, X[3], range(n_rows)))
    # and the next good call is clean
    ok_n = torch.tensor([n_rows], dtype=torch.int32, device=DEV)
    B.lif_sparse_ffn_static(gpu.cache, n_rows, bias, X[3], None, ok_n, b_down, got, cfg.d_model)
    assert B.lif_sparse_ffn_static_status() == B.LIF_OK
    gpu.close()


def test_static_scratch_ffn_rejects_sizes_beyond_its_array():
    x = torch.zeros(16384, dtype=torch.float16, device=DEV)
    y = torch.zeros(16384, dtype=torch.float32, device=DEV)
    n = torch.zeros(1, dtype=torch.int32, device=DEV)
    for d_bad in (8200, 16384, 12, 0):
        with pytest.raises(B.LifError) as e:
            B.lif_sparse_ffn_static(x, 1, x, x, None, n, None, y, d_bad)
        assert e.value.code == B.LIF_ERR_INVALID_ARG
    with pytest.raises(B.LifError) as e:
        B.lif_sparse_ffn_static(x, 0, x, x, None, n, None, y, 256)
    assert e.value.code == B.LIF_ERR_INVALID_ARG
    with pytest.raises(B.LifError) as e:
        B.lif_sparse_ffn_static(x, 1, x, x[1:], None, n, None, y, 256)
    assert e.value.code == B.LIF_ERR_ALIGNMENT
