"""What the library does with input it must not trust and with waits that run out — checked
on the GPU in forms that cannot fault: a bad row index is replaced before it is used as an
address, a damaged snapshot is refused on the host, and a wait is made to run out by giving it
no polls at all while the copies it guards still land before the kernel returns."""
import numpy as np
import pytest
import torch

from oracle import lif_oracle as O
from paper_2312_11514_b200 import binding as B
from paper_2312_11514_b200 import workloads as W

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _warm_layer(S, steps=4, **kw):
    cfg = W.LifConfig("guards", 1, 1032, 4096, 32, 3, S, 8, 0.10, 1.0, 0.8, 0.6, 33)
    gpu, ora = P.make_layer_pair(cfg, 0, b_down=True, **kw)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(S, cfg.d_model, dtype=torch.float32, device=DEV)
    for t in range(steps):
        B.lif_decode_step(gpu.handle, X[t], y)
        P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
    return cfg, gpu, ora, X, y


def _own_rows_reference(gpu, x, rows):
    """Oracle FFN (float64) over rows of the GPU's own cache and bias arrays."""
    matrix = gpu.cache.cpu().numpy()
    bias = gpu._view("bias", gpu.capacity, torch.float16).cpu().numpy()
    return O.sparse_ffn(matrix, bias, np.asarray(rows, dtype=np.int64), x.cpu().numpy(),
                        gpu.keep["bias_down"].cpu().numpy())


@pytest.mark.parametrize("S", [1, 4])
def test_sparse_ffn_never_addresses_a_row_outside_the_cache(S):
    cfg, gpu, ora, X, y = _warm_layer(S)
    cap = gpu.capacity
    rows = [3, cap, 9, -1, cap - 1, 2 ** 30, 0, -(2 ** 31)]     # cap - 1 and 0: the valid ends
    valid = [r for r in rows if 0 <= r < cap]
    slots = torch.tensor(rows, dtype=torch.int32, device=DEV)
    n = torch.tensor([len(rows)], dtype=torch.int32, device=DEV)
    B.lif_sparse_ffn(gpu.handle, X[5], slots, n, y)
    st = B.lif_get_stats(gpu.handle)
    assert st.status == B.LIF_ERR_INVALID_ARG
    P.assert_y_close(y.cpu().numpy().astype(np.float64), _own_rows_reference(gpu, X[5], valid))
    # a count beyond the cache is clamped to it (rows [0, capacity))
    B.lif_clear_status(gpu.handle)
    B.lif_sparse_ffn(gpu.handle, X[5], None, torch.tensor([cap + 77], dtype=torch.int32, device=DEV), y)
    assert B.lif_get_stats(gpu.handle).status == B.LIF_ERR_INVALID_ARG
    P.assert_y_close(y.cpu().numpy().astype(np.float64), _own_rows_reference(gpu, X[5], range(cap)))
    # a negative count is no rows
    B.lif_clear_status(gpu.handle)
    B.lif_sparse_ffn(gpu.handle, X[5], None, torch.tensor([-5], dtype=torch.int32, device=DEV), y)
    assert B.lif_get_stats(gpu.handle).status == B.LIF_ERR_INVALID_ARG
    want = np.tile(gpu.keep["bias_down"].float().cpu().numpy(), (S, 1))
    np.testing.assert_array_equal(y.cpu().numpy(), want)
    # the layer itself is unharmed: clear, and the next token follows the oracle again
    B.lif_clear_status(gpu.handle)
    B.lif_decode_step(gpu.handle, X[4], y)
    P.check_decode_step(gpu, ora, X[4].cpu().numpy(), y)
    gpu.close()


@pytest.mark.parametrize("S", [1, 4])
def test_a_wait_that_runs_out_is_reported_and_leaves_the_layer_usable(S):
    cfg, gpu, ora, X, y = _warm_layer(S)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    # no polls at all on the first wait of every copy: the CTA flags the timeout at once, then
    # waits for its copies with the full limit, so nothing is left in flight when it returns
    B.lif_set_tuning(gpu.handle, B.TUNE_WAIT_POLLS, 0)
    B.lif_decode_step(gpu.handle, X[4], y, sc, sf)
    g = gpu.lists()
    assert g["status"] == B.LIF_ERR_TIMEOUT
    # the window update of that step ran before the FFN and follows the oracle
    lists = ora.cache.window_update(g["active_idx"])
    ora.cache.insert(lists, ora.bundles, ora.bias_up)
    for key in P.LIST_KEYS:
        np.testing.assert_array_equal(g[key], lists[key], err_msg=key)
    np.testing.assert_array_equal(g["pointers"], ora.cache.pointers)
    np.testing.assert_array_equal(g["last_active"], ora.cache.last_active)
    P.compare_cache_rows(gpu, ora)
    # while the status stands, further window updates are refused: nothing moves
    B.lif_set_tuning(gpu.handle, B.TUNE_WAIT_POLLS, 1 << 22)
    B.lif_decode_step(gpu.handle, X[5], y, sc, sf)
    g2 = gpu.lists()
    assert g2["status"] == B.LIF_ERR_TIMEOUT and g2["step"] == g["step"]
    np.testing.assert_array_equal(g2["pointers"], g["pointers"])
    np.testing.assert_array_equal(g2["last_active"], g["last_active"])
    assert len(g2["load_ids"]) == 0 and len(g2["evict_ids"]) == 0
    # cleared, the same token goes through and matches the oracle
    B.lif_clear_status(gpu.handle)
    B.lif_decode_step(gpu.handle, X[5], y, sc, sf)
    P.check_decode_step(gpu, ora, X[5].cpu().numpy(), y)
    with pytest.raises(B.LifError):
        B.lif_set_tuning(gpu.handle, B.TUNE_WAIT_POLLS, -1)
    gpu.close()


def test_staged_ffn_with_a_wait_that_runs_out():
    cfg, gpu, ora, X, y = _warm_layer(1)
    F = gpu.d_ff
    B.lif_set_tuning(gpu.handle, B.TUNE_WAIT_POLLS, 0)
    B.lif_sparse_ffn(gpu.handle, X[3], gpu._view("active_slots", F), gpu.counts[B.CNT_N_ACTIVE:], y)
    assert B.lif_get_stats(gpu.handle).status == B.LIF_ERR_TIMEOUT
    B.lif_set_tuning(gpu.handle, B.TUNE_WAIT_POLLS, 1 << 22)
    B.lif_clear_status(gpu.handle)
    B.lif_sparse_ffn(gpu.handle, X[3], gpu._view("active_slots", F), gpu.counts[B.CNT_N_ACTIVE:], y)
    g = gpu.lists()
    assert g["status"] == B.LIF_OK
    P.assert_y_close(y.cpu().numpy().astype(np.float64), _own_rows_reference(gpu, X[3], g["active_slots"]))
    gpu.close()


def test_restore_refuses_a_damaged_snapshot_on_the_host():
    cfg, gpu, ora, X, y = _warm_layer(1)
    snap = B.lif_snapshot(gpu.handle)
    before = gpu.lists()
    cap, F = gpu.capacity, gpu.d_ff
    words = np.frombuffer(snap, dtype=np.int32, count=B.CNT_LEN + cap + 2 * F).copy()
    ptr0, so0, la0 = B.CNT_LEN, B.CNT_LEN + cap, B.CNT_LEN + cap + F
    n = int(words[B.CNT_NUM_USED])
    assert n > 10

    def damaged(edit):
        w = words.copy()
        edit(w)
        return w.tobytes() + bytes(snap[w.nbytes:])

    some_cached = int(words[ptr0 + 2])
    free_id = int(np.nonzero(words[so0:so0 + F] < 0)[0][0])
    cases = {
        "row names no neuron": lambda w: w.__setitem__(ptr0 + 1, -1),
        "row names a neuron beyond d_ff": lambda w: w.__setitem__(ptr0 + 1, F),
        "two rows name one neuron": lambda w: w.__setitem__(ptr0 + 1, some_cached),
        "neuron points at another row": lambda w: w.__setitem__(so0 + some_cached, 5),
        "absent neuron claims a row": lambda w: w.__setitem__(so0 + free_id, 0),
        "free row not marked free": lambda w: w.__setitem__(ptr0 + n, 3),
        "row count beyond the rows in use": lambda w: w.__setitem__(B.CNT_NUM_USED, n + 1),
        "row count negative": lambda w: w.__setitem__(B.CNT_NUM_USED, -1),
        "stamp from the future": lambda w: w.__setitem__(la0 + some_cached, int(w[B.CNT_STEP]) + 3),
        "negative step": lambda w: w.__setitem__(B.CNT_STEP, -2),
    }
    for name, edit in cases.items():
        with pytest.raises(B.LifError) as e:
            B.lif_restore(gpu.handle, damaged(edit))
        assert e.value.code == B.LIF_ERR_STATE, name
    after = gpu.lists()                      # nothing reached the device
    for key in ("pointers", "slot_of", "last_active"):
        np.testing.assert_array_equal(before[key], after[key])
    B.lif_restore(gpu.handle, snap)          # the intact one is still accepted
    B.lif_decode_step(gpu.handle, X[4], y)
    P.check_decode_step(gpu, ora, X[4].cpu().numpy(), y)
    gpu.close()


def test_guard_row_and_guard_block_survive_a_run_that_fills_the_cache():
    # a threshold below every score makes all neurons active: the first step loads d_ff bundles
    # into a cache of exactly d_ff rows, every list of the workspace is filled to its last
    # element, and nothing is written past the cache or the workspace
    cfg = W.LifConfig("full", 1, 264, 512, 16, 4, 1, 4, 0.30, 0.3, 0.5, 0.6, 5)
    gpu, ora = P.make_layer_pair(cfg, 0, capacity=cfg.d_ff, theta=-1e30, b_down=True)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for t in range(cfg.steps):
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        lists = P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
        assert lists["num_used"] == cfg.d_ff and len(lists["active_slots"]) == cfg.d_ff
        assert gpu.guards_intact()
    assert len(gpu.lists()["hit_slots"]) == cfg.d_ff
    gpu.close()          # raises if a guard was touched


@pytest.mark.parametrize("gate_mode", [B.GATE_NONE, B.GATE_RESIDENT])
def test_predictor_calls_between_steps_do_not_leak_into_the_next_step(gate_mode):
    # lif_predict with another input leaves the predictor's masks (which the fetch kernel of a
    # decode step reads while that step's predictor may still be running) describing neurons the
    # step does not want; every step must still bring in exactly its own
    cfg = W.LifConfig("between", 1, 520, 4096, 32, 3, 1, 14, 0.08, 1.0, 0.8, 0.6, 41)
    kw = dict(gate_mode=gate_mode, b_down=True)
    if gate_mode == B.GATE_RESIDENT:
        kw.update(activation=B.ACT_FATRELU, act_threshold=0.05)
    gpu, ora = P.make_layer_pair(cfg, 0, **kw)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(1, cfg.d_model, dtype=torch.float32, device=DEV)
    idx = torch.empty(cfg.d_ff, dtype=torch.int32, device=DEV)
    n = torch.zeros(1, dtype=torch.int32, device=DEV)
    sc, sf = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for t in range(cfg.steps):
        other = X[(t + 5) % cfg.steps]
        for _ in range(1 + t % 3):
            B.lif_predict(gpu.handle, other, None, idx, n, sc)
        B.lif_decode_step(gpu.handle, X[t], y, sc, sf)
        P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
        P.compare_cache_rows(gpu, ora)
    gpu.close()
