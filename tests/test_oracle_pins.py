"""Pins for the CPU oracle: each part is checked against something other than itself —
textbook definitions written as brute-force loops, closed forms, set-history brute force, and
the numbers the paper prints."""
import math
import os

import numpy as np
import pytest

from oracle import lif_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "cost_model_paper_values.txt")


def _rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ predictor
def test_predictor_matches_scalar_loops():
    r = _rng(0)
    S, d, k, F = 2, 7, 3, 11
    x, A, B, c = r.normal(size=(S, d)), r.normal(size=(d, k)), r.normal(size=(k, F)), r.normal(size=F)
    got = O.predictor_logits(x, A, B, c)
    for s in range(S):
        for i in range(F):
            acc = 0.0
            for j in range(k):
                z = 0.0
                for m in range(d):
                    z += x[s, m] * A[m, j]
                acc += z * B[j, i]
            assert got[s, i] == pytest.approx(acc + c[i], rel=1e-12, abs=1e-12)


def test_predictor_rank_one_closed_form():
    # A = u (d x 1), B = v^T (1 x F): score_i = (x.u) v_i + c_i
    r = _rng(1)
    d, F = 13, 9
    x, u, v, c = r.normal(size=(1, d)), r.normal(size=(d, 1)), r.normal(size=(1, F)), r.normal(size=F)
    got = O.predictor_logits(x, u, v, c)[0]
    want = float(x[0] @ u[:, 0]) * v[0] + c
    np.testing.assert_allclose(got, want, rtol=1e-12)


def test_predictor_identity_factors_select_coordinates():
    # A = I, B = [I | 0]: score_i = x_i + c_i for i < d, c_i beyond — catches transposes.
    d, F = 5, 8
    x = np.arange(1.0, d + 1)[None, :]
    B = np.zeros((d, F)); B[:, :d] = np.eye(d)
    c = 10.0 * np.arange(F)
    got = O.predictor_logits(x, np.eye(d), B, c)[0]
    want = c.copy(); want[:d] += x[0]
    np.testing.assert_array_equal(got, want)


def test_active_set_strict_threshold_and_stream_union():
    logits = np.array([[0.0, 1.0, -1.0, 0.5, 0.0],
                       [0.5, -2.0, -1.0, 0.5, 0.0]])
    np.testing.assert_array_equal(O.active_set(logits, 0.0), [0, 1, 3])      # == theta inactive
    np.testing.assert_array_equal(O.active_set(logits[:1], 0.0), [1, 3])
    np.testing.assert_array_equal(O.active_set(logits, 0.75), [1])
    assert O.active_set(logits, np.inf).size == 0
    assert O.active_set(logits, -np.inf).size == 5


def test_sigmoid_threshold():
    assert O.sigmoid_threshold_to_logit(0.5) == 0.0
    for tau in (0.4, 0.7):                       # thresholds used in Appendix B
        th = O.sigmoid_threshold_to_logit(tau)
        assert 1.0 / (1.0 + math.exp(-th)) == pytest.approx(tau, rel=1e-12)


# ------------------------------------------------------------------ sparse FFN
def _dense_ffn_loops(W_up, b_up, W_down, x, b_down):
    F, d = W_up.shape
    y = [b_down[m] for m in range(d)]
    for i in range(F):
        pre = b_up[i]
        for m in range(d):
            pre += W_up[i, m] * x[m]
        if pre > 0.0:
            for m in range(d):
                y[m] += pre * W_down[m, i]
    return np.array(y)


def _cache_from_dense(W_up, b_up, W_down, ids, cap=None):
    F, d = W_up.shape
    cap = cap or len(ids)
    M = np.zeros((cap, 2 * d)); bias = np.zeros(cap)
    for s, i in enumerate(ids):
        M[s, :d] = W_up[i]; M[s, d:] = W_down[:, i]; bias[s] = b_up[i]
    return M, bias


def test_sparse_ffn_with_true_mask_equals_dense_ffn():
    r = _rng(2)
    F, d = 23, 6
    W_up, W_down = r.normal(size=(F, d)), r.normal(size=(d, F))
    b_up, b_down, x = r.normal(size=F), r.normal(size=d), r.normal(size=d)
    dense = _dense_ffn_loops(W_up, b_up, W_down, x, b_down)
    true_active = [i for i in range(F) if W_up[i] @ x + b_up[i] > 0]
    assert 0 < len(true_active) < F
    M, bias = _cache_from_dense(W_up, b_up, W_down, true_active)
    got = O.sparse_ffn(M, bias, np.arange(len(true_active)), x[None, :], b_down)[0]
    np.testing.assert_allclose(got, dense, rtol=1e-12, atol=1e-12)
    # every neuron cached (theta = -inf): ReLU zeroes the rest, still the dense FFN
    M, bias = _cache_from_dense(W_up, b_up, W_down, list(range(F)))
    got = O.sparse_ffn(M, bias, np.arange(F), x[None, :], b_down)[0]
    np.testing.assert_allclose(got, dense, rtol=1e-12, atol=1e-12)
    # library form of the same textbook definition
    lib = W_down @ np.maximum(W_up @ x + b_up, 0) + b_down
    np.testing.assert_allclose(got, lib, rtol=1e-12, atol=1e-12)


def test_sparse_ffn_row_order_and_empty_and_streams():
    r = _rng(3)
    F, d, S = 12, 5, 3
    W_up, W_down = r.normal(size=(F, d)), r.normal(size=(d, F))
    b_up, b_down, X = r.normal(size=F), r.normal(size=d), r.normal(size=(S, d))
    ids = [7, 2, 9, 4]
    M, bias = _cache_from_dense(W_up, b_up, W_down, ids, cap=6)
    y0 = O.sparse_ffn(M, bias, [0, 1, 2, 3], X, b_down)
    perm = [2, 0, 3, 1]                                    # Section 3.3 item 3: order-free
    M2, bias2 = M.copy(), bias.copy()
    M2[:4], bias2[:4] = M[perm], bias[perm]
    np.testing.assert_allclose(O.sparse_ffn(M2, bias2, [0, 1, 2, 3], X, b_down), y0, rtol=1e-12)
    np.testing.assert_allclose(O.sparse_ffn(M, bias, [3, 1, 0, 2], X, b_down), y0, rtol=1e-12)
    # no active rows: only the down bias is left; without it, zeros
    np.testing.assert_array_equal(O.sparse_ffn(M, bias, [], X, b_down), np.tile(b_down, (S, 1)))
    np.testing.assert_array_equal(O.sparse_ffn(M, bias, [], X), np.zeros((S, d)))
    # streams are independent rows
    for s in range(S):
        np.testing.assert_allclose(O.sparse_ffn(M, bias, [0, 1, 2, 3], X[s:s + 1], b_down)[0], y0[s],
                                   rtol=1e-12)
    # a subset of the slots is the dense FFN restricted to those neurons
    sub = O.sparse_ffn(M, bias, [1, 3], X[:1], None)[0]
    want = sum(max(W_up[i] @ X[0] + b_up[i], 0.0) * W_down[:, i] for i in (2, 4))
    np.testing.assert_allclose(sub, want, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ window protocol
def _random_active_sets(F, T, rate, seed, sticky=0.6):
    r = _rng(seed)
    pop = np.clip(rate * np.exp(r.normal(size=F)), 0, 0.9)
    prev = np.zeros(F, dtype=bool)
    out = []
    for _ in range(T):
        cur = (r.random(F) < pop) | (prev & (r.random(F) < sticky * 0.5))
        out.append(np.nonzero(cur)[0].astype(np.int32))
        prev = cur
    return out


def _check_structure(cache):
    n = cache.num_used
    ptr = cache.pointers[:n]
    assert len(set(ptr.tolist())) == n and (ptr >= 0).all()
    for s in range(n):
        assert cache.slot_of[ptr[s]] == s
    assert (cache.slot_of >= 0).sum() == n
    assert (cache.pointers[n:] == -1).all()


@pytest.mark.parametrize("k", [1, 2, 5])
def test_window_matches_set_history_brute_force(k):
    F, d, T = 97, 4, 40
    r = _rng(10 + k)
    bundles = r.normal(size=(F, 2 * d)).astype(np.float16)
    bias_up = r.normal(size=F).astype(np.float16)
    sets = _random_active_sets(F, T, 0.08, seed=k)
    cache = O.NeuronCache(d, F, capacity=F, window_k=k)
    total_loaded = 0
    for t, act in enumerate(sets):
        before = cache.cached_ids()
        n_before = cache.num_used
        rows_before = {int(cache.pointers[s]): cache.matrix[s].copy() for s in range(n_before)}
        slot_before = cache.slot_of.copy()
        lists = cache.window_update(act)
        cache.insert(lists, bundles, bias_up)
        _check_structure(cache)
        # cached set = union of the active sets of the last k tokens, current included
        union = set()
        for u in range(max(0, t - k + 1), t + 1):
            union |= set(sets[u].tolist())
        assert cache.cached_ids() == union
        # load = needed but absent, ascending; evict = present but outside the window
        assert lists["load_ids"].tolist() == sorted(set(act.tolist()) - before)
        assert set(lists["evict_ids"].tolist()) == before - union
        assert cache.num_used == n_before - len(lists["evict_ids"]) + len(lists["load_ids"])
        # new rows are stacked at the end: rows num_kept .. num_kept + num_new
        n_kept = n_before - len(lists["evict_ids"])
        assert lists["load_slots"].tolist() == list(range(n_kept, n_kept + len(lists["load_ids"])))
        # deleting rewrites at most one row per deleted neuron, only from the tail into holes
        assert len(lists["move_src"]) <= len(lists["evict_ids"])
        assert all(src >= n_kept > dst for src, dst in zip(lists["move_src"], lists["move_dst"]))
        moved = {int(cache.pointers[dst]) for dst in lists["move_dst"]}
        for i in before & union:
            if i not in moved:
                assert cache.slot_of[i] == slot_before[i]          # untouched rows stay put
        # every cached row holds exactly its neuron's bundle and bias
        for s in range(cache.num_used):
            i = cache.pointers[s]
            np.testing.assert_array_equal(cache.matrix[s], bundles[i])
            assert cache.bias[s] == bias_up[i]
            if i in rows_before:
                np.testing.assert_array_equal(cache.matrix[s], rows_before[i])
        # slot lists handed to the FFN
        assert [int(cache.pointers[s]) for s in lists["active_slots"]] == act.tolist()
        assert sorted(lists["hit_slots"].tolist() + lists["load_slots"].tolist()) == \
            sorted(lists["active_slots"].tolist())
        total_loaded += len(lists["load_ids"])
        assert cache.bytes_fetched == total_loaded * 2 * d * 2     # |new| x bundle bytes
    if k == 1:
        # window of one token: load = A_t \ A_{t-1}
        c2 = O.NeuronCache(d, F, F, 1)
        prev = set()
        for act in sets:
            ls = c2.window_update(act)
            assert ls["load_ids"].tolist() == sorted(set(act.tolist()) - prev)
            prev = set(act.tolist())


def test_window_longer_than_sequence_never_evicts_and_growth_slows():
    F, T = 400, 30
    sets = _random_active_sets(F, T, 0.05, seed=5, sticky=0.0)
    cache = O.NeuronCache(2, F, F, window_k=T + 1)
    used = []
    for act in sets:
        ls = cache.window_update(act)
        assert ls["evict_ids"].size == 0 and ls["move_src"].size == 0
        used.append(cache.num_used)
    assert used[-1] == len(set(np.concatenate(sets).tolist()))
    inc = np.diff([0] + used)
    # aggregated usage is concave on average (Section 3.1, aggregated neuron usage figure)
    assert inc[: T // 2].mean() > inc[T // 2:].mean()


def test_window_swap_remove_worked_example():
    # rows [10 11 12 13 14 15]; neurons 11, 14 and 15 leave the window, nothing new arrives.
    # Holes below the new size: slot 1.  Last surviving row (slot 3, neuron 13) fills it.
    F, d = 32, 2
    cache = O.NeuronCache(d, F, 8, window_k=1)
    bundles = np.arange(F * 2 * d, dtype=np.float16).reshape(F, 2 * d)
    bias_up = np.arange(F, dtype=np.float16)
    ls = cache.window_update([10, 11, 12, 13, 14, 15]); cache.insert(ls, bundles, bias_up)
    assert cache.pointers[:6].tolist() == [10, 11, 12, 13, 14, 15]
    ls = cache.window_update([10, 12, 13]); cache.insert(ls, bundles, bias_up)
    assert ls["evict_ids"].tolist() == [11, 14, 15]
    assert ls["move_src"].tolist() == [3] and ls["move_dst"].tolist() == [1]
    assert cache.pointers[:3].tolist() == [10, 13, 12] and cache.num_used == 3
    np.testing.assert_array_equal(cache.matrix[1], bundles[13])
    assert cache.bias[1] == bias_up[13]
    assert ls["active_slots"].tolist() == [0, 2, 1]
    # two holes, two tail survivors: the very last survivor fills the first hole
    cache = O.NeuronCache(d, F, 8, window_k=1)
    ls = cache.window_update([1, 2, 3, 4, 5, 6]); cache.insert(ls, bundles, bias_up)
    ls = cache.window_update([3, 4, 5, 6, 20]); cache.insert(ls, bundles, bias_up)
    assert ls["move_src"].tolist() == [5, 4] and ls["move_dst"].tolist() == [0, 1]
    assert cache.pointers[:5].tolist() == [6, 5, 3, 4, 20]
    assert ls["load_ids"].tolist() == [20] and ls["load_slots"].tolist() == [4]
    assert ls["hit_slots"].tolist() == [2, 3, 1, 0]


def test_window_capacity_error_leaves_state_unchanged():
    cache = O.NeuronCache(2, 16, capacity=4, window_k=2)
    cache.window_update([0, 1, 2])
    snap = (cache.pointers.copy(), cache.slot_of.copy(), cache.last_active.copy(), cache.num_used, cache.t)
    with pytest.raises(O.CapacityError):
        cache.window_update([3, 4])
    assert (cache.pointers == snap[0]).all() and (cache.slot_of == snap[1]).all()
    assert (cache.last_active == snap[2]).all() and (cache.num_used, cache.t) == snap[3:]
    cache.window_update([3])                                         # exactly fills: fine
    assert cache.num_used == 4


def test_cold_start_loads_whole_active_set():
    # the first tokens find an empty cache (Section 4, long-generation figure)
    cache = O.NeuronCache(2, 50, 50, window_k=3)
    ls = cache.window_update([4, 8, 15, 16, 23, 42])
    assert ls["load_ids"].tolist() == [4, 8, 15, 16, 23, 42]
    assert ls["load_slots"].tolist() == list(range(6)) and ls["hit_slots"].size == 0


# ------------------------------------------------------------------ decode step
def test_decode_step_with_true_mask_predictor_equals_dense_ffn():
    # A predictor that reproduces the up projection exactly (A = W_up^T, B = I, c = b_up)
    # predicts the true ReLU mask, so every step's output is the dense FFN, whatever the
    # cache did in between.
    r = _rng(7)
    F, d, T = 40, 8, 12
    W_up = r.normal(size=(F, d)).astype(np.float16)
    W_down = r.normal(size=(d, F)).astype(np.float16)
    b_up = (r.normal(size=F) - 1.0).astype(np.float16)
    bundles = np.concatenate([W_up, W_down.T], axis=1)
    cache = O.NeuronCache(d, F, F, window_k=3)
    x = r.normal(size=(1, d))
    for _ in range(T):
        x = (0.8 * x + 0.6 * r.normal(size=(1, d))).astype(np.float16)
        _, act, lists, y = O.decode_step(cache, x, W_up.T, np.eye(F), b_up, 0.0, bundles, b_up)
        xd = x[0].astype(np.float64)
        dense = W_down.astype(np.float64) @ np.maximum(W_up.astype(np.float64) @ xd + b_up, 0.0)
        np.testing.assert_allclose(y[0], dense, rtol=1e-10, atol=1e-10)
        # the whole-cache mode adds only rows whose ReLU is zero or that really fire: same y
        y_all = O.sparse_ffn(cache.matrix, cache.bias, np.arange(cache.num_used), x)
        np.testing.assert_allclose(y_all[0], dense, rtol=1e-10, atol=1e-10)


# ------------------------------------------------------------------ cost model
def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            kind, inputs, value, tol, cite = [p.strip() for p in line.split("|")]
            rows.append((kind, inputs, float(value), float(tol), cite))
    return rows


@pytest.mark.parametrize("kind,inputs,value,tol,cite", _golden_rows())
def test_cost_model_reproduces_paper_values(kind, inputs, value, tol, cite):
    if kind == "io_ms":
        gb, thr = map(float, inputs.split(","))
        got = O.io_latency_ms(gb, thr)
    elif kind == "chunk_bytes":
        d, nb = map(int, inputs.split(","))
        got = O.chunk_bytes(d, nb)
        assert O.chunk_bytes(d, nb, bundled=False) * 2 == got          # bundling doubles it
    elif kind == "dram_share":
        fixed, ffn, frac = inputs.split(";")
        got = O.dram_share_percent([float(v) for v in fixed.split(",")], float(ffn), float(frac))
    elif kind == "flash_gb":
        got = O.flash_to_dram_gb(*map(float, inputs.split(",")))
    elif kind == "avg_rank":
        n1, r1, n2, r2 = map(float, inputs.split(","))
        got = O.average_predictor_rank([n1, n2], [r1, r2])
    elif kind == "predictor_fraction":
        got = O.predictor_weight_fraction(*map(int, inputs.split(",")))
    elif kind == "kv_fraction":
        ctx, d, L, params = inputs.split(",")
        got = O.kv_cache_fraction(int(ctx), int(d), int(L), float(params))
    else:
        raise AssertionError(kind)
    assert got == pytest.approx(value, rel=tol, abs=0), cite


def test_bundling_halves_io_latency_as_in_table_1():
    # same bytes, throughput 1.25 -> 2.25 GB/s: latency ratio 164 / 87 in Table 1
    a, b = O.io_latency_ms(0.2, 1.25), O.io_latency_ms(0.2, 2.25)
    assert a / b == pytest.approx(164 / 87, rel=0.05)


# ------------------------------------------------------------------ activation variants
@pytest.mark.parametrize("activation,threshold", [(O.RELU_SQUARED, 0.0), (O.FATRELU, 0.7), (O.FATRELU, 0.0)])
def test_activation_variants_match_scalar_loops(activation, threshold):
    r = _rng(20 + activation)
    F, d = 17, 5
    W_up, W_down = r.normal(size=(F, d)), r.normal(size=(d, F))
    b_up, b_down, x = r.normal(size=F), r.normal(size=d), r.normal(size=d)
    want = b_down.copy()
    n_pass = 0
    for i in range(F):
        pre = b_up[i] + sum(W_up[i, m] * x[m] for m in range(d))
        if activation == O.RELU_SQUARED:
            h = pre * pre if pre > 0 else 0.0            # Appendix C, Persimmon: squared ReLU
        else:
            h = pre if pre > threshold else 0.0          # Appendix C, Llama 2: FATReLU
        n_pass += h != 0.0
        for m in range(d):
            want[m] += h * W_down[m, i]
    assert 0 < n_pass < F
    M, bias = _cache_from_dense(W_up, b_up, W_down, list(range(F)))
    got = O.sparse_ffn(M, bias, np.arange(F), x[None, :], b_down, activation, threshold)[0]
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)
    if activation == O.FATRELU and threshold == 0.0:     # threshold 0 is plain ReLU
        np.testing.assert_allclose(got, O.sparse_ffn(M, bias, np.arange(F), x[None, :], b_down)[0], rtol=1e-12)


def test_fatrelu_threshold_only_removes_neurons():
    pre = np.array([-1.0, 0.2, 0.7, 0.70001, 3.0])
    np.testing.assert_array_equal(O.activation_fn(pre, O.FATRELU, 0.7), [0, 0, 0, 0.70001, 3.0])
    np.testing.assert_array_equal(O.activation_fn(pre, O.RELU_SQUARED), [0, 0.2 ** 2, 0.7 ** 2, 0.70001 ** 2, 9.0])
    np.testing.assert_array_equal(O.activation_fn(pre), [0, 0.2, 0.7, 0.70001, 3.0])


# ------------------------------------------------------------------ memory-budgeted window
def test_budgeted_window_brute_force():
    # Appendix C (Persimmon 8B, Phi-2): the window shrinks whenever the cache would pass the
    # budget.  Brute force from the stored history of active sets and of what was cached.
    F, T, k, budget = 300, 60, 5, 70
    sets = _random_active_sets(F, T, 0.07, seed=31, sticky=0.3)
    cache = O.NeuronCache(2, F, capacity=F, window_k=k, budget_rows=budget)
    free = O.NeuronCache(2, F, capacity=F, window_k=k)
    last_seen = {}
    shrunk = 0
    for t, act in enumerate(sets):
        before = cache.cached_ids()
        lists = cache.window_update(act)
        free.window_update(act)
        for i in act.tolist():
            last_seen[i] = t
        ke = lists["k_eff"]
        assert 1 <= ke <= k
        kept_expected = lambda kk: {i for i in before | set(act.tolist()) if last_seen[i] > t - kk}
        assert cache.cached_ids() == kept_expected(ke)                  # exactly the k'-window
        assert cache.num_used <= budget
        if ke < k:                                                      # widest that fits
            shrunk += 1
            assert len(kept_expected(ke + 1)) > budget
        assert set(act.tolist()) <= cache.cached_ids() <= free.cached_ids()
        _check_structure(cache)
    assert 5 < shrunk < T                                               # the budget really binds
    # a budget nothing ever reaches changes nothing
    a, b = O.NeuronCache(2, F, F, k, budget_rows=F), O.NeuronCache(2, F, F, k)
    for act in sets[:20]:
        la, lb = a.window_update(act), b.window_update(act)
        assert la["k_eff"] == k
        for key in ("evict_ids", "move_src", "load_ids", "active_slots"):
            np.testing.assert_array_equal(la[key], lb[key])


def test_budget_smaller_than_active_set_is_refused_unchanged():
    cache = O.NeuronCache(2, 64, capacity=64, window_k=3, budget_rows=8)
    cache.window_update(np.arange(6, dtype=np.int32))
    snap = (cache.pointers.copy(), cache.last_active.copy(), cache.num_used, cache.t)
    with pytest.raises(O.CapacityError):
        cache.window_update(np.arange(20, 30, dtype=np.int32))           # 10 active > budget 8
    assert (cache.pointers == snap[0]).all() and (cache.last_active == snap[1]).all()
    assert (cache.num_used, cache.t) == snap[2:]
    ls = cache.window_update(np.arange(20, 27, dtype=np.int32))          # 7 fit once the window is 1
    assert ls["k_eff"] == 1 and cache.num_used == 7


# ------------------------------------------------------------------ multi-token window update
def _pass_info(sets, F, keep):
    """Union and keep_token of a pass given its per-token active sets."""
    union = sorted(set().union(*[set(a.tolist()) for a in sets]))
    kt = [max([j for j in range(keep) if i in set(sets[j].tolist())], default=-1) for i in union]
    return np.array(union, dtype=np.int32), np.array(kt)


def test_multi_token_update_equals_sequential_updates_when_everything_is_kept():
    # a pass of S <= k consecutive tokens, all kept: same cached set and same stamps as S
    # single-token updates (Section 4, speculative decoding: the window is updated with
    # several tokens at once)
    F, k = 200, 5
    sets = _random_active_sets(F, 24, 0.06, seed=41)
    for S in (1, 2, 4):
        multi, single = O.NeuronCache(2, F, F, k), O.NeuronCache(2, F, F, k)
        for p in range(0, 24, S):
            chunk = sets[p:p + S]
            act, kt = _pass_info(chunk, F, S)
            ls = multi.window_update(act, kt, keep=S)
            for a in chunk:
                single.window_update(a)
            assert multi.t == single.t == p + S
            assert multi.cached_ids() == single.cached_ids()
            np.testing.assert_array_equal(multi.last_active, single.last_active)
            assert [int(multi.pointers[s]) for s in ls["active_slots"]] == act.tolist()
            _check_structure(multi)


def test_multi_token_update_keeps_the_window_ending_at_the_kept_token():
    # 5 tokens per pass (lambda = 4), keep the window ending with token m of the pass:
    # brute force from the history of kept tokens
    F, k, S, m = 300, 3, 5, 2
    sets = _random_active_sets(F, 40, 0.05, seed=43)
    cache = O.NeuronCache(2, F, F, k)
    kept_history = []                                    # active sets of the kept tokens, in time order
    for p in range(0, 40, S):
        chunk = sets[p:p + S]
        act, kt = _pass_info(chunk, F, m)
        before = cache.cached_ids()
        ls = cache.window_update(act, kt, keep=m)
        kept_history += [set(a.tolist()) for a in chunk[:m]]
        window = set().union(*kept_history[-k:])
        needed_now = set(act.tolist())
        assert cache.cached_ids() == (before & window) | needed_now | (window & needed_now)
        assert cache.cached_ids() == ((before | needed_now) & window) | needed_now
        assert cache.t == len(kept_history)
        assert ls["load_ids"].tolist() == sorted(needed_now - before)
        # a neuron active only beyond the kept token is dropped by the next pass unless needed again
        late_only = needed_now - set().union(*[set(a.tolist()) for a in chunk[:m]]) - (before & window)
        if p + S < 40:
            nxt = sets[p + S:p + 2 * S]
            act2, kt2 = _pass_info(nxt, F, m)
            probe = O.NeuronCache(2, F, F, k)
            probe.__dict__.update({k_: (v.copy() if isinstance(v, np.ndarray) else v)
                                   for k_, v in cache.__dict__.items()})
            probe.window_update(act2, kt2, keep=m)
            assert not (late_only - set(act2.tolist())) & probe.cached_ids()
        _check_structure(cache)


def _clone_cache(cache):
    twin = O.NeuronCache(cache.d_model, cache.d_ff, cache.capacity, cache.k)
    twin.__dict__.update({k_: (v.copy() if isinstance(v, np.ndarray) else v)
                          for k_, v in cache.__dict__.items()})
    return twin


@pytest.mark.parametrize("k,S,m", [(2, 5, 5), (2, 5, 4), (3, 5, 5), (1, 4, 3), (3, 8, 7), (2, 5, 2)])
def test_multi_token_pass_longer_than_the_window(k, S, m):
    # A pass that keeps more tokens than the window holds (m > k; Section 4, "Speculative
    # Decoding": the window is updated with several tokens at once).  Everything is derived
    # from the per-token history, nothing from the oracle's stamp expression:
    #   cached set  = neurons active in the last k kept tokens, plus every neuron the pass used
    #                 (a pass does not delete what it uses);
    #   window invariant in stamp form (Section 3.1): cached  <=>  last_active > t - k;
    #   horizon     = with no further activity a cached neuron leaves at the first single-token
    #                 step whose window no longer holds a kept token in which it was active,
    #                 and not before the step after the pass that used it.
    # Invariant and horizon together leave one value for each stamp: horizon - k.
    F = 240
    T = 6 * S
    sets = _random_active_sets(F, T, 0.05, seed=100 + 10 * k + m)
    cache = O.NeuronCache(2, F, F, k)
    kept = []                                    # (time, active set) of every kept token
    for p in range(0, T, S):
        chunk = sets[p:p + S]
        act, kt = _pass_info(chunk, F, m)
        before = cache.cached_ids()
        ls = cache.window_update(act, kt, keep=m)
        t0 = len(kept)
        kept += [(t0 + j, set(chunk[j].tolist())) for j in range(m)]
        t = len(kept) - 1                        # time of the kept token that ends the window
        assert cache.t == t + 1
        used = set(act.tolist())
        in_window = set().union(*[a for (tau, a) in kept if tau > t - k])
        expect = (before & in_window) | used
        assert cache.cached_ids() == expect
        assert ls["load_ids"].tolist() == sorted(used - before)
        assert set(ls["evict_ids"].tolist()) == before - expect
        # window invariant in stamp form
        by_stamp = set(np.nonzero(cache.last_active > t - k)[0].tolist())
        assert by_stamp == expect
        # horizon of every cached neuron, by brute force over the kept history
        last_kept = {i: max([tau for (tau, a) in kept if i in a], default=None) for i in expect}
        horizon = {i: max(t + 1, (last_kept[i] + k) if last_kept[i] is not None else t + 1)
                   for i in expect}
        probe = _clone_cache(cache)
        left_at = {}
        for step in range(t + 1, t + k + 2):     # empty single-token steps
            gone = probe.cached_ids()
            probe.window_update(np.zeros(0, dtype=np.int32))
            gone -= probe.cached_ids()
            for i in gone:
                left_at[i] = step
        assert left_at == horizon
        for i in expect:
            assert cache.last_active[i] == horizon[i] - k
        _check_structure(cache)


def test_stamps_of_a_long_pass_worked_example():
    # k = 2, one pass of 5 kept tokens (times 0..4).  Neuron 7 is active in token 0 only,
    # neuron 8 in token 3, neuron 9 in token 4, neuron 6 in tokens 1 and 3.  The window after
    # the pass is {3, 4}.  7 was used by the pass, so it is still cached, but no token of the
    # window holds it: it must leave at the very next step, i.e. carry the oldest stamp of the
    # window (3); 6 and 8 carry 3, 9 carries 4.
    cache = O.NeuronCache(2, 16, 16, 2)
    act = np.array([6, 7, 8, 9], dtype=np.int32)
    cache.window_update(act, np.array([3, 0, 3, 4]), keep=5)
    assert cache.t == 5 and cache.cached_ids() == {6, 7, 8, 9}
    assert cache.last_active[[6, 7, 8, 9]].tolist() == [3, 3, 3, 4]
    cache.window_update(np.zeros(0, dtype=np.int32))         # time 5: window {4, 5}
    assert cache.cached_ids() == {9}
    cache.window_update(np.zeros(0, dtype=np.int32))         # time 6: window {5, 6}
    assert cache.cached_ids() == set()


def test_keep_tokens_helper():
    logits = np.array([[1.0, -1, -1, 1], [-1, 1.0, -1, 1], [-1, -1, 1.0, -1]])
    act = O.active_set(logits, 0.0)
    assert act.tolist() == [0, 1, 2, 3]
    assert O.keep_tokens(logits, 0.0, act, 3).tolist() == [0, 1, 2, 1]
    assert O.keep_tokens(logits, 0.0, act, 2).tolist() == [0, 1, -1, 1]
    assert O.keep_tokens(logits, 0.0, act, 1).tolist() == [0, -1, -1, 0]


# ------------------------------------------------------------------ gated FFN (Appendix C, Llama 2)
def _gated_loops(W_gate, b_gate, W_up, W_down, x, b_down, activation, threshold):
    """Textbook gated FFN, scalar loops: y = W_down (act(W_gate x + b) * (W_up x)) + b_down."""
    F, d = W_gate.shape
    y = [b_down[m] for m in range(d)]
    n_pass = 0
    for i in range(F):
        g = b_gate[i] + sum(W_gate[i, m] * x[m] for m in range(d))
        u = sum(W_up[i, m] * x[m] for m in range(d))
        if activation == O.FATRELU:
            a = g if g > threshold else 0.0
        elif activation == O.RELU_SQUARED:
            a = g * g if g > 0 else 0.0
        else:
            a = g if g > 0 else 0.0
        n_pass += a != 0.0
        for m in range(d):
            y[m] += a * u * W_down[m, i]
    return np.array(y), n_pass


def _gated_cache(W_gate, b_gate, W_up, W_down, ids):
    F, d = W_gate.shape
    M = np.zeros((len(ids), 3 * d)); bias = np.zeros(len(ids))
    for s, i in enumerate(ids):
        M[s, :d] = W_gate[i]; M[s, d:2 * d] = W_up[i]; M[s, 2 * d:] = W_down[:, i]; bias[s] = b_gate[i]
    return M, bias


@pytest.mark.parametrize("activation,threshold", [(O.FATRELU, 0.4), (O.RELU, 0.0), (O.RELU_SQUARED, 0.0)])
def test_gated_ffn_matches_scalar_loops_and_library_form(activation, threshold):
    r = _rng(40 + activation)
    F, d, S = 19, 6, 2
    W_gate, W_up, W_down = r.normal(size=(F, d)), r.normal(size=(F, d)), r.normal(size=(d, F))
    b_gate, b_down, X = r.normal(size=F) * 0.3, r.normal(size=d), r.normal(size=(S, d))
    order = r.permutation(F)                                  # rows in any order
    M, bias = _gated_cache(W_gate, b_gate, W_up, W_down, order)
    got = O.sparse_ffn(M, bias, np.arange(F), X, b_down, activation, threshold, gated=True)
    for s in range(S):
        want, n_pass = _gated_loops(W_gate, b_gate, W_up, W_down, X[s], b_down, activation, threshold)
        assert 0 < n_pass < F
        np.testing.assert_allclose(got[s], want, rtol=1e-12, atol=1e-12)
    lib = (O.activation_fn(X @ W_gate.T + b_gate, activation, threshold) * (X @ W_up.T)) @ W_down.T + b_down
    np.testing.assert_allclose(got, lib, rtol=1e-12, atol=1e-12)
    # only the neurons whose gate passes matter: dropping the others changes nothing
    passing = [q for q in range(F)
               if (O.activation_fn(X @ M[q, :d] + bias[q], activation, threshold) != 0).any()]
    np.testing.assert_allclose(O.sparse_ffn(M, bias, np.array(passing), X, b_down, activation, threshold,
                                            gated=True), got, rtol=1e-12, atol=1e-12)


def test_gated_ffn_special_cases_reduce_to_the_plain_ffn():
    r = _rng(44)
    F, d = 15, 5
    W_gate, W_down = r.normal(size=(F, d)), r.normal(size=(d, F))
    b_down, x = r.normal(size=d), r.normal(size=d)
    zero = np.zeros(F)
    # up row == gate row, no bias, ReLU: relu(g) * g is the squared ReLU of the plain FFN
    M3, bias3 = _gated_cache(W_gate, zero, W_gate, W_down, list(range(F)))
    M2, bias2 = _cache_from_dense(W_gate, zero, W_down, list(range(F)))
    np.testing.assert_allclose(O.sparse_ffn(M3, bias3, np.arange(F), x[None], b_down, O.RELU, gated=True),
                               O.sparse_ffn(M2, bias2, np.arange(F), x[None], b_down, O.RELU_SQUARED),
                               rtol=1e-12, atol=1e-12)
    # up rows with <up_i, x> = 1: the gate value passes through, i.e. the plain FFN (with its bias)
    b_gate = r.normal(size=F)
    W_one = np.tile(x / (x @ x), (F, 1))
    M3, bias3 = _gated_cache(W_gate, b_gate, W_one, W_down, list(range(F)))
    M2, bias2 = _cache_from_dense(W_gate, b_gate, W_down, list(range(F)))
    np.testing.assert_allclose(O.sparse_ffn(M3, bias3, np.arange(F), x[None], b_down, O.FATRELU, 0.3, gated=True),
                               O.sparse_ffn(M2, bias2, np.arange(F), x[None], b_down, O.FATRELU, 0.3),
                               rtol=1e-11, atol=1e-12)
    # the activation acts on the gate only: exchanging gate and up rows changes the result
    W_up = r.normal(size=(F, d))
    Ma, ba = _gated_cache(W_gate, zero, W_up, W_down, list(range(F)))
    Mb, bb = _gated_cache(W_up, zero, W_gate, W_down, list(range(F)))
    ya = O.sparse_ffn(Ma, ba, np.arange(F), x[None], None, O.RELU, gated=True)
    yb = O.sparse_ffn(Mb, bb, np.arange(F), x[None], None, O.RELU, gated=True)
    assert np.abs(ya - yb).max() > 1e-3
    # empty list
    np.testing.assert_array_equal(O.sparse_ffn(Ma, ba, np.array([], dtype=np.int64), x[None], b_down, gated=True)[0], b_down)


def test_gate_projection_as_predictor_reproduces_the_dense_gated_ffn_at_every_step():
    """With the resident gate as predictor the active set is exactly the set of neurons with a
    non-zero activation, so every step's output is the dense gated FFN, whatever the window."""
    r = _rng(45)
    F, d, S, k, thr = 40, 6, 2, 3, 0.5
    W_gate, W_up, W_down = r.normal(size=(F, d)), r.normal(size=(F, d)), r.normal(size=(d, F))
    b_gate, b_down = r.normal(size=F) * 0.2 - 0.8, r.normal(size=d)
    bundles = np.concatenate([W_up, W_down.T], axis=1).astype(np.float16)     # up | down
    Wg16, bg16 = W_gate.astype(np.float16), b_gate.astype(np.float16)
    cache = O.NeuronCache(d, F, F, k)
    history, n_loaded = [], 0
    for t in range(10):
        X = r.normal(size=(S, d)).astype(np.float16)
        g, act, lists, y = O.decode_step_gate_predictor(cache, X, Wg16, bg16, bundles, b_down,
                                                        activation=O.FATRELU, threshold=thr)
        for s in range(S):
            want, _ = _gated_loops(Wg16.astype(float), bg16.astype(float), bundles[:, :d].astype(float),
                                   bundles[:, d:].astype(float).T, X[s].astype(float), b_down, O.FATRELU, thr)
            np.testing.assert_allclose(y[s], want, rtol=1e-11, atol=1e-12)
        # score = gate pre-activation (scalar loop on a few entries); active = passes for some stream
        for i in (0, 7, F - 1):
            assert abs(g[1, i] - (float(bg16[i]) + sum(float(Wg16[i, m]) * float(X[1, m]) for m in range(d)))) < 1e-12
        assert act.tolist() == [i for i in range(F) if (g[:, i] > thr).any()]
        history.append(set(act.tolist()))
        n_loaded += len(lists["load_ids"])
        assert cache.cached_ids() == set().union(*history[-k:])
        assert 0 < len(act) < F
        # whole-cache FFN gives the same result: cached, inactive rows have a zero activation
        ids = cache.pointers[:cache.num_used]
        yw = O.sparse_ffn(cache.matrix, cache.bias, np.arange(cache.num_used), X, b_down, O.FATRELU, thr,
                          gate_pre=g[:, ids])
        np.testing.assert_allclose(yw, y, rtol=1e-11, atol=1e-12)
    assert cache.bytes_fetched == n_loaded * 2 * d * 2          # two vectors per bundle: the gate stays resident
    assert cache.matrix.shape[1] == 2 * d


def test_gated_decode_step_three_vector_bundles():
    """Low-rank predictor + three-vector bundles: with a predictor that is exact for the gate
    (rank d: A = I, B = W_gate^T, c = b_gate, theta = threshold) a step equals the dense gated
    FFN, and the traffic is 6*d bytes per new neuron."""
    r = _rng(46)
    F, d, k, thr = 30, 5, 2, 0.3
    W_gate, W_up, W_down = (r.normal(size=(F, d)).astype(np.float16), r.normal(size=(F, d)).astype(np.float16),
                            r.normal(size=(d, F)).astype(np.float16))
    b_gate = (r.normal(size=F) * 0.2 - 0.5).astype(np.float16)
    bundles = np.concatenate([W_gate, W_up, W_down.T], axis=1)
    cache = O.NeuronCache(d, F, F, k, n_vec=3)
    n_loaded = 0
    for t in range(8):
        x = r.normal(size=(1, d)).astype(np.float16)
        logits, act, lists, y = O.decode_step(cache, x, np.eye(d), W_gate.astype(float).T, b_gate.astype(float),
                                              thr, bundles, b_gate, activation=O.FATRELU, threshold=thr, gated=True)
        want, n_pass = _gated_loops(W_gate.astype(float), b_gate.astype(float), W_up.astype(float),
                                    W_down.astype(float), x[0].astype(float), np.zeros(d), O.FATRELU, thr)
        assert n_pass == len(act)
        np.testing.assert_allclose(y[0], want, rtol=1e-11, atol=1e-12)
        n_loaded += len(lists["load_ids"])
    assert cache.bytes_fetched == n_loaded * 3 * d * 2 and n_loaded > 0
    assert cache.matrix.shape == (F, 3 * d)


# ------------------------------------------------------------------ append first, then delete
@pytest.mark.parametrize("k", [1, 2, 5])
def test_append_first_window_brute_force(k):
    """Section 3.3 with its two operations in the other order (stack the new neurons, then
    delete by pulling last rows into freed ones): same cached set, traffic and outputs as the
    paper's order; new neurons land in freed rows; old rows move only when more are deleted
    than arrive."""
    F, d, T = 97, 4, 40
    r = _rng(70 + k)
    bundles = r.normal(size=(F, 2 * d)).astype(np.float16)
    bias_up = r.normal(size=F).astype(np.float16)
    sets = _random_active_sets(F, T, 0.08, seed=k)
    cache = O.NeuronCache(d, F, capacity=F, window_k=k, append_first=True)
    paper = O.NeuronCache(d, F, capacity=F, window_k=k)
    saw_reuse = saw_append = saw_move = False
    for t, act in enumerate(sets):
        before = cache.cached_ids()
        n = cache.num_used
        slot_before = cache.slot_of.copy()
        rows_before = {int(cache.pointers[s]): cache.matrix[s].copy() for s in range(n)}
        freed = sorted(int(cache.slot_of[i]) for i in before
                       if i not in set(act.tolist()) and cache.last_active[i] <= t - k)
        lists = cache.window_update(act)
        cache.insert(lists, bundles, bias_up)
        ref = paper.window_update(act)
        paper.insert(ref, bundles, bias_up)
        _check_structure(cache)
        union = set()
        for u in range(max(0, t - k + 1), t + 1):
            union |= set(sets[u].tolist())
        assert cache.cached_ids() == union == paper.cached_ids()
        for key in ("load_ids", "evict_ids"):
            assert sorted(lists[key].tolist()) == sorted(ref[key].tolist())
        e, l = len(freed), len(lists["load_ids"])
        assert cache.num_used == n - e + l == paper.num_used
        # brute-force statement of the placement: the last min(e, l) new neurons take the freed
        # rows, lowest freed row <- highest id; the other new neurons stay stacked at n, n+1, ...
        want = [n + j if j < l - min(e, l) else freed[l - 1 - j] for j in range(l)]
        assert lists["load_slots"].tolist() == want
        # old rows move only when deletions outnumber arrivals, never more than the paper's order
        assert len(lists["move_src"]) <= max(0, e - l) and len(lists["move_src"]) <= len(ref["move_src"])
        b = n - max(0, e - l)
        assert all(src >= b > dst and dst in freed[min(e, l):] for src, dst in zip(lists["move_src"], lists["move_dst"]))
        assert lists["move_src"].tolist() == sorted(lists["move_src"].tolist(), reverse=True)   # last row first
        assert lists["move_dst"].tolist() == sorted(lists["move_dst"].tolist())
        moved = {int(cache.pointers[dst]) for dst in lists["move_dst"]}
        for i in before & union:
            if i not in moved:
                assert cache.slot_of[i] == slot_before[i]
        for s in range(cache.num_used):
            i = cache.pointers[s]
            np.testing.assert_array_equal(cache.matrix[s], bundles[i])
            assert cache.bias[s] == bias_up[i]
            if i in rows_before:
                np.testing.assert_array_equal(cache.matrix[s], rows_before[i])
        assert [int(cache.pointers[s]) for s in lists["active_slots"]] == act.tolist()
        assert sorted(lists["hit_slots"].tolist() + lists["load_slots"].tolist()) == \
            sorted(lists["active_slots"].tolist())
        # the FFN does not see the row order
        x = r.normal(size=(1, d))
        np.testing.assert_allclose(O.sparse_ffn(cache.matrix, cache.bias, lists["active_slots"], x),
                                   O.sparse_ffn(paper.matrix, paper.bias, ref["active_slots"], x),
                                   rtol=1e-12, atol=1e-12)
        saw_reuse |= l > 0 and e > 0
        saw_append |= l > e
        saw_move |= len(lists["move_src"]) > 0
    assert cache.bytes_fetched == paper.bytes_fetched and cache.rows_moved < paper.rows_moved
    assert saw_reuse and saw_append and saw_move


def test_append_first_worked_example_and_transient_overshoot():
    # 6 rows cached (neurons 10..15 in rows 0..5), capacity 7.  Rows 1 and 4 are deleted and the
    # neurons 3, 7, 20 arrive: stacked they would stand in rows 6, 7, 8 (beyond the capacity for a
    # moment); the deletions pull 20 into row 1 and 7 into row 4; 3 stays in row 6.
    cache = O.NeuronCache(2, 32, capacity=7, window_k=1, append_first=True)
    cache.window_update(np.arange(10, 16))
    lists = cache.window_update(np.array([3, 7, 10, 12, 13, 15, 20]))
    assert lists["evict_ids"].tolist() == [11, 14]
    assert lists["load_ids"].tolist() == [3, 7, 20] and lists["load_slots"].tolist() == [6, 4, 1]
    assert lists["move_src"].size == 0
    assert cache.pointers.tolist() == [10, 20, 12, 13, 7, 15, 3] and cache.num_used == 7
    # more deletions than arrivals: 20, 12 and 3 go, 11 arrives.  Stacked, 11 stands in row 7 and
    # goes to the first freed row (1); then the last row still in use, row 5 (15), goes to row 2;
    # row 6 was freed itself and is dropped with the tail
    lists = cache.window_update(np.array([7, 10, 11, 13, 15]))
    assert sorted(lists["evict_ids"].tolist()) == [3, 12, 20]
    assert lists["load_ids"].tolist() == [11] and lists["load_slots"].tolist() == [1]
    assert lists["move_src"].tolist() == [5] and lists["move_dst"].tolist() == [2]
    assert cache.pointers.tolist() == [10, 11, 15, 13, 7, -1, -1] and cache.num_used == 5
    # capacity still refuses what does not fit at the end of the step
    with pytest.raises(O.CapacityError):
        cache.window_update(np.arange(0, 9))


def test_append_first_agrees_with_the_papers_order_under_budget_and_multi_token_updates():
    # the order of the two cache operations changes rows, never sets, window choices or traffic
    F, d, T = 120, 3, 40
    r = _rng(90)
    bundles = r.normal(size=(F, 2 * d)).astype(np.float16)
    bias_up = r.normal(size=F).astype(np.float16)
    sets = _random_active_sets(F, T, 0.10, seed=9)
    a = O.NeuronCache(d, F, F, window_k=5, budget_rows=34, append_first=True)
    b = O.NeuronCache(d, F, F, window_k=5, budget_rows=34)
    ks = []
    for act in sets:
        la, lb = a.window_update(act), b.window_update(act)
        a.insert(la, bundles, bias_up); b.insert(lb, bundles, bias_up)
        _check_structure(a)
        assert la["k_eff"] == lb["k_eff"] and a.cached_ids() == b.cached_ids()
        assert sorted(la["evict_ids"].tolist()) == sorted(lb["evict_ids"].tolist())
        assert la["load_ids"].tolist() == lb["load_ids"].tolist() and a.num_used <= 34
        ks.append(la["k_eff"])
    assert min(ks) < 5 and a.bytes_fetched == b.bytes_fetched and a.rows_moved <= b.rows_moved
    # several tokens per update (speculative decoding), window ending at the second token
    a = O.NeuronCache(d, F, F, window_k=3, append_first=True)
    b = O.NeuronCache(d, F, F, window_k=3)
    for t in range(0, T - 4, 4):
        logits = np.full((4, F), -1.0)
        for j in range(4):
            logits[j, sets[t + j]] = 1.0
        act = O.active_set(logits, 0.0)
        kt = O.keep_tokens(logits, 0.0, act, 2)
        la, lb = a.window_update(act, kt, 2), b.window_update(act, kt, 2)
        a.insert(la, bundles, bias_up); b.insert(lb, bundles, bias_up)
        _check_structure(a)
        assert a.cached_ids() == b.cached_ids() and a.t == b.t
        np.testing.assert_array_equal(a.last_active, b.last_active)
        for s in range(a.num_used):
            np.testing.assert_array_equal(a.matrix[s], bundles[a.pointers[s]])


# ------------------------------------------------------------------ neuron sharding
def test_neuron_shard_ranges_tile_the_ids():
    for F, G in ((24, 1), (24, 2), (24, 3), (1024, 8)):
        ranges = [O.neuron_shard_range(F, g, G) for g in range(G)]
        assert ranges[0][0] == 0 and ranges[-1][1] == F
        assert all(a[1] == b[0] for a, b in zip(ranges, ranges[1:]))
        assert len({hi - lo for lo, hi in ranges}) == 1
    with pytest.raises(ValueError):
        O.neuron_shard_range(10, 0, 3)
    with pytest.raises(ValueError):
        O.neuron_shard_range(12, 3, 3)


@pytest.mark.parametrize("G", [2, 4])
def test_sharded_step_with_true_mask_predictor_equals_dense_ffn(G):
    # Same construction as the single-device pin: the predictor reproduces the up projection,
    # so the summed partial outputs must equal the dense FFN (bias of the down projection
    # added once, not once per device) at every step.
    r = _rng(70 + G)
    F, d, T = 48, 8, 10
    W_up = r.normal(size=(F, d)).astype(np.float16)
    W_down = r.normal(size=(d, F)).astype(np.float16)
    b_up = (r.normal(size=F) - 1.0).astype(np.float16)
    b_down = r.normal(size=d).astype(np.float16)
    bundles = np.concatenate([W_up, W_down.T], axis=1)
    caches = [O.NeuronCache(d, F // G, F // G, window_k=3) for _ in range(G)]
    x = r.normal(size=(1, d))
    for _ in range(T):
        x = (0.8 * x + 0.6 * r.normal(size=(1, d))).astype(np.float16)
        _, y = O.sharded_decode_step(caches, x, W_up.T, np.eye(F), b_up, 0.0, bundles, b_up, b_down)
        xd = x[0].astype(np.float64)
        dense = W_down.astype(np.float64) @ np.maximum(W_up.astype(np.float64) @ xd + b_up, 0.0)
        np.testing.assert_allclose(y[0], dense + b_down, rtol=1e-10, atol=1e-10)


@pytest.mark.parametrize("G,append_first", [(1, False), (2, False), (3, True)])
def test_sharded_step_partitions_the_single_device_step(G, append_first):
    # Random low-rank predictor: the devices' active lists, cached sets and fetched bytes
    # partition those of one device holding every neuron, and the partial outputs sum to its
    # output.  One shard is the single-device step itself, bit for bit.
    r = _rng(80 + G)
    F, d, rank, S, T, k = 60, 16, 4, 2, 14, 3
    bundles = r.normal(scale=0.3, size=(F, 2 * d)).astype(np.float16)
    bias_up = r.normal(scale=0.2, size=F).astype(np.float16)
    A = r.normal(size=(d, rank)).astype(np.float16)
    B = r.normal(size=(rank, F)).astype(np.float16)
    c = (r.normal(size=F) - 1.2).astype(np.float32)
    b_down = r.normal(size=d).astype(np.float16)
    one = O.NeuronCache(d, F, F, window_k=k, append_first=append_first)
    caches = [O.NeuronCache(d, F // G, F // G, window_k=k, append_first=append_first) for _ in range(G)]
    x = r.normal(size=(S, d))
    for _ in range(T):
        x = (0.7 * x + 0.7 * r.normal(size=(S, d))).astype(np.float16)
        logits, act, lists, y_one = O.decode_step(one, x, A, B, c, 0.0, bundles, bias_up, b_down)
        parts, y = O.sharded_decode_step(caches, x, A, B, c, 0.0, bundles, bias_up, b_down)
        if G == 1:
            np.testing.assert_array_equal(y, y_one)
            np.testing.assert_array_equal(parts[0][2]["load_slots"], lists["load_slots"])
        np.testing.assert_allclose(y, y_one, rtol=1e-11, atol=1e-11)
        got_act, got_cached = [], set()
        for g, (lg, a, _, _) in enumerate(parts):
            lo, hi = O.neuron_shard_range(F, g, G)
            np.testing.assert_array_equal(lg, logits[:, lo:hi])
            got_act.extend((a + lo).tolist())
            got_cached |= {i + lo for i in caches[g].cached_ids()}
        assert got_act == act.tolist()
        assert got_cached == one.cached_ids()
        assert sum(ch.bytes_fetched for ch in caches) == one.bytes_fetched
        assert sum(ch.num_used for ch in caches) == one.num_used
