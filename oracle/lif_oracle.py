"""CPU oracle for the per-token, per-FFN-layer path of "LLM in a flash" (arXiv 2312.11514).

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, deliberately unoptimised statement of
what the method computes, in float64 over the fp16-stored values.  It shares no code with the
CUDA library and is imported only by the tests, the smoke check and the benchmark's CPU
baseline.  The product never calls it.

Per decode step and per layer (paper Sections 3.1-3.3):

1. low-rank predictor: scores = x.A.B + c, neuron i is *active* iff score_i > theta
   (Section 3.1 "Anticipating ReLU Sparsity", Section 3.1 "The Sliding Window Technique":
   an active neuron is one with a positive predictor output; Appendix B uses a sigmoid
   threshold tau, which in the logit domain is theta = ln(tau / (1 - tau)));
2. sliding window over the last k tokens: neurons not predicted active in any of the last k
   tokens (the current one included) are deleted, newly needed ones are loaded
   (Section 3.1 "The Sliding Window Technique");
3. cache management (Section 3.3): rows to delete are overwritten by the last rows so the
   used rows stay consecutive, new rows are stacked at the end
   (rows num_used .. num_used + num_new);
4. inference (Section 3.3 item 3): matrix[:, :d_model] is the up projection and
   matrix[:, d_model:] transposed is the down projection of the cached neurons.

Parity pins (tests marked "not gpu"): dense brute force for the FFN, pure-Python loops and
rank-1 closed forms for the predictor, brute-force set history for the window protocol, and
the numbers the paper prints for the cost model (tests/golden/).  The *order* of rows inside
the cache is a convention the paper only draws in a figure: "parity unpinned" for the slot
order itself (only its invariants are pinned); everything that depends on it (FFN output,
cached set, bytes fetched) is order-independent and pinned.
"""
from __future__ import annotations

import numpy as np

NEVER = -(2 ** 30)          # "never predicted active" stamp


# --------------------------------------------------------------------------------------
# Step 1: low-rank predictor (Section 3.1; Appendix B)
# --------------------------------------------------------------------------------------
def predictor_logits(x, A, B, c):
    """scores[s][i] = sum_j (sum_m x[s][m] A[m][j]) B[j][i] + c[i], float64.

    x: [S][d], A: [d][r], B: [r][F], c: [F].  Two bias-free linear maps with no
    non-linearity between them, plus a per-neuron offset."""
    x = np.asarray(x, dtype=np.float64)
    z = x @ np.asarray(A, dtype=np.float64)              # [S][r]
    return z @ np.asarray(B, dtype=np.float64) + np.asarray(c, dtype=np.float64)[None, :]


def active_set(logits, theta):
    """Ascending ids of the neurons whose score exceeds theta for at least one stream
    (score == theta is inactive)."""
    mask = (np.asarray(logits) > theta).any(axis=0)
    return np.nonzero(mask)[0].astype(np.int32)


def keep_tokens(logits, theta, act, keep):
    """For a pass of consecutive tokens (rows of ``logits``): the last token j < keep in which
    each neuron of ``act`` is active, -1 if none."""
    m = np.asarray(logits)[:keep, :][:, act] > theta          # [keep][n_act]
    last = np.where(m.any(axis=0), keep - 1 - np.argmax(m[::-1], axis=0), -1)
    return last.astype(np.int64)


def sigmoid_threshold_to_logit(tau):
    """theta = ln(tau / (1 - tau)); tau = 0.5 is the "positive output" rule."""
    return float(np.log(tau / (1.0 - tau)))


# --------------------------------------------------------------------------------------
# Steps 2-4: the preallocated neuron cache (Section 3.3)
# --------------------------------------------------------------------------------------
class CapacityError(Exception):
    pass


class NeuronCache:
    """matrix / pointers / bias / num_used / last_k_active of Section 3.3.

    ``last_k_active`` is kept as ``last_active[i]`` = the last step at which neuron i was
    predicted active, so "still inside the window of k tokens" is last_active[i] > t - k."""

    def __init__(self, d_model, d_ff, capacity, window_k, budget_rows=0, n_vec=2,
                 append_first=False):
        """``budget_rows`` > 0 turns on the memory budget of Appendix C (Persimmon 8B, Phi-2):
        whenever the cache would pass the budget, the window is shrunk for that step.
        ``n_vec`` = vectors of d_model values per bundle: 2 (up row, down column; Section 3.2)
        or 3 for a gated FFN (gate row, up row, down column; Appendix C, Llama 2).
        ``append_first`` applies the two operations of Section 3.3 in the other order: the new
        neurons are stacked at the end first (item 2), then the deletions pull the last rows
        into the freed ones (item 1) -- so a new neuron that would be moved straight away is
        written into the freed row directly and only the deletions that outnumber the
        arrivals move old rows.  Same cached set, different row order."""
        self.d_model, self.d_ff, self.capacity, self.k = d_model, d_ff, capacity, window_k
        self.budget_rows = budget_rows
        self.n_vec = n_vec
        self.append_first = append_first
        self.k_eff = window_k
        self.matrix = np.zeros((capacity, n_vec * d_model), dtype=np.float16)
        self.pointers = np.full(capacity, -1, dtype=np.int32)
        self.bias = np.zeros(capacity, dtype=np.float16)
        self.slot_of = np.full(d_ff, -1, dtype=np.int32)
        self.last_active = np.full(d_ff, NEVER, dtype=np.int32)
        self.num_used = 0
        self.t = 0
        self.bytes_fetched = 0
        self.rows_moved = 0

    # -- delete + plan ------------------------------------------------------------------
    def window_update(self, act, keep_token=None, keep=1):
        """One window step for the ascending active list ``act``.  Deletes the neurons that
        left the window (Section 3.3 item 1), and assigns rows to the ones to bring in
        (item 2).  Returns the lists; the new rows' weights arrive with ``insert``.

        Speculative decoding (Section 4, "Speculative Decoding"): the pass holds several
        consecutive tokens and the window is updated with all of them at once, keeping the
        last k tokens that end with token ``keep`` of the pass.  ``act`` is then the union
        over the pass and ``keep_token[q]`` the last token j < keep in which neuron act[q] is
        active, or -1 if it is active only in later tokens: such a neuron is needed for this
        pass but does not enter the kept window, so it gets the oldest stamp still inside it
        (as does a neuron whose kept token is already older than the window).
        Time advances by ``keep`` tokens."""
        act = np.asarray(act, dtype=np.int32)
        k, n = self.k, self.num_used
        if keep_token is None:
            keep_token = np.zeros(len(act), dtype=np.int64)
        keep_token = np.asarray(keep_token, dtype=np.int64)
        assert keep >= 1 and len(keep_token) == len(act) and (keep_token < keep).all()
        assert keep == 1 or self.budget_rows == 0
        t0 = self.t
        t = t0 + keep - 1                       # the kept window ends at this token
        in_act = np.zeros(self.d_ff, dtype=bool)
        in_act[act] = True

        # what would be deleted / loaded, before anything is changed
        load_ids = [int(i) for i in act if self.slot_of[i] < 0]

        def would_evict(kk):
            return [s for s in range(n)
                    if not in_act[self.pointers[s]]
                    and self.last_active[self.pointers[s]] <= t - kk]

        evict_slots = would_evict(k)
        limit = self.capacity
        if self.budget_rows > 0:
            # Memory budget: keep the widest window k' <= k whose rows, with the rows to
            # bring in, fit the budget; the choice is made anew at every step.
            limit = min(limit, self.budget_rows)
            while k > 1 and n - len(evict_slots) + len(load_ids) > limit:
                k -= 1
                evict_slots = would_evict(k)
        n_new = n - len(evict_slots)
        if n_new + len(load_ids) > limit:
            raise CapacityError(f"need {n_new + len(load_ids)} rows, have {limit}")
        self.k_eff = k

        # no neuron used by this pass is deleted by it: stamps never fall below the oldest
        # one still inside the kept window (only matters when the pass is longer than k)
        stamps = np.maximum(np.where(keep_token >= 0, t0 + keep_token, self.last_active[act]),
                            t - self.k + 1)
        self.last_active[act] = stamps
        evict_ids = [int(self.pointers[s]) for s in evict_slots]

        # With append_first the rows to bring in already stand at the end (rows n .. n + n_load,
        # ascending neuron id) when the deletions are applied; their weights are not there yet,
        # so "moving" one of them only decides where its bundle will be written.
        n_load = len(load_ids)
        end = n
        ptr = np.concatenate([self.pointers, np.full(n_load, -1, dtype=np.int32)])   # room to stack
        if self.append_first:
            ptr[n:n + n_load] = load_ids
            self.slot_of[load_ids] = np.arange(n, n + n_load)
            end = n + n_load

        # Deleting: walk the freed rows in ascending order; the current last row replaces
        # the freed one unless the last row is itself to be deleted, in which case it is
        # simply dropped.
        dead = np.zeros(len(ptr), dtype=bool)
        dead[evict_slots] = True
        for i in evict_ids:
            self.slot_of[i] = -1
        move_src, move_dst = [], []
        tail = end
        for hole in evict_slots:
            while tail > 0 and dead[tail - 1]:
                tail -= 1                                   # drop deleted rows off the end
            if hole >= tail:
                break                                       # every remaining hole was dropped
            tail -= 1                                       # last surviving row
            ptr[hole] = ptr[tail]
            self.slot_of[ptr[hole]] = hole
            dead[hole] = False
            if tail < n:                                    # a cached row: its weights move
                self.matrix[hole] = self.matrix[tail]
                self.bias[hole] = self.bias[tail]
                move_src.append(tail)
                move_dst.append(hole)
        self.rows_moved += len(move_src)
        n_new = n - len(evict_slots)                        # rows left of the old ones

        if self.append_first:
            load_slots = [int(self.slot_of[i]) for i in load_ids]
        else:
            # Bringing in new neurons: rows num_used .. num_used + num_new, ascending neuron id.
            load_slots = list(range(n_new, n_new + n_load))
            for i, s in zip(load_ids, load_slots):
                ptr[s] = i
                self.slot_of[i] = s
        self.num_used = n_new + n_load
        ptr[self.num_used:] = -1
        self.pointers[:] = ptr[:self.capacity]
        self.t = t0 + keep

        active_slots = self.slot_of[act].astype(np.int32)
        hit_slots = active_slots[~np.isin(act, np.asarray(load_ids, dtype=np.int32))]
        i32 = lambda v: np.asarray(v, dtype=np.int32)
        return {
            "evict_ids": i32(evict_ids), "move_src": i32(move_src), "move_dst": i32(move_dst),
            "load_ids": i32(load_ids), "load_slots": i32(load_slots),
            "active_slots": active_slots, "hit_slots": i32(hit_slots),
            "num_used_before": n, "num_kept": n_new, "num_used": self.num_used,
            "k_eff": self.k_eff,
        }

    # -- insert -------------------------------------------------------------------------
    def insert(self, lists, bundles, bias_up):
        """Copy the bundles of the newly needed neurons from the full store into their rows,
        and their up-projection biases (resident scalars) into ``bias`` (Section 3.3 item 2)."""
        for i, s in zip(lists["load_ids"], lists["load_slots"]):
            self.matrix[s] = bundles[i]
            self.bias[s] = bias_up[i]
        self.bytes_fetched += len(lists["load_ids"]) * self.n_vec * self.d_model * self.matrix.itemsize

    def cached_ids(self):
        return set(int(i) for i in self.pointers[: self.num_used])


# --------------------------------------------------------------------------------------
# Step 5: sparse FFN over the cached bundles (Section 3.3 item 3)
# --------------------------------------------------------------------------------------
RELU, RELU_SQUARED, FATRELU = 0, 1, 2


def activation_fn(pre, activation=RELU, threshold=0.0):
    """The FFN non-linearities the paper runs: ReLU (OPT, relufied Falcon and Phi-2), squared
    ReLU (Appendix C, Persimmon 8B) and FATReLU (Appendix C, Llama 2: a neuron passes its
    pre-activation only when it exceeds a threshold)."""
    if activation == RELU:
        return np.maximum(pre, 0.0)
    if activation == RELU_SQUARED:
        return np.maximum(pre, 0.0) ** 2
    if activation == FATRELU:
        return np.where(pre > threshold, pre, 0.0)
    raise ValueError(activation)


def sparse_ffn(matrix, bias, slots, x, b_down=None, activation=RELU, threshold=0.0,
               gated=False, gate_pre=None):
    """y[s] = b_down + sum_q act(<matrix[slots[q], :d], x[s]> + bias[slots[q]]) * matrix[slots[q], d:]

    matrix: [cap][2d] (fp16 values), bias: [cap], slots: row indices, x: [S][d].  float64.

    ``gated`` (Appendix C, Llama 2: a gated linear unit, an up and a down projection, the
    activation applied to the gate value): rows are [cap][3d] = gate | up | down and
    y[s] = b_down + sum_q act(<gate_q, x[s]> + bias_q) * <up_q, x[s]> * down_q.

    ``gate_pre`` [S][len(slots)] (Appendix C, Llama 2, "alternative approaches": the gate
    projection stays resident and doubles as the predictor): the gate pre-activations of the
    rows are given, rows are [cap][2d] = up | down, ``bias`` is not used:
    y[s] = b_down + sum_q act(gate_pre[s][q]) * <up_q, x[s]> * down_q."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[1]
    rows = np.asarray(matrix)[np.asarray(slots, dtype=np.int64)].astype(np.float64)
    assert rows.shape[1] == (3 if gated else 2) * d and not (gated and gate_pre is not None)
    first, down = rows[:, :d], rows[:, -d:]
    if gate_pre is not None:
        h = activation_fn(np.asarray(gate_pre, dtype=np.float64), activation, threshold) * (x @ first.T)
    else:
        h = activation_fn(x @ first.T + np.asarray(bias, dtype=np.float64)[slots][None, :],
                          activation, threshold)
        if gated:
            h = h * (x @ rows[:, d:2 * d].T)
    y = h @ down
    if b_down is not None:
        y = y + np.asarray(b_down, dtype=np.float64)[None, :]
    return y


def gate_scores(x, gate_matrix, gate_bias=None):
    """Gate pre-activations of every neuron, g[s][i] = <gate_matrix[i], x[s]> + gate_bias[i]:
    with the gate projection resident they are the predictor's scores, and a neuron is active
    iff its gate value passes the activation's threshold (Appendix C, Llama 2)."""
    g = np.asarray(x, dtype=np.float64) @ np.asarray(gate_matrix, dtype=np.float64).T
    if gate_bias is not None:
        g = g + np.asarray(gate_bias, dtype=np.float64)[None, :]
    return g


def decode_step(cache, x, A, B, c, theta, bundles, bias_up, b_down=None, whole_cache=False,
                act=None, activation=RELU, threshold=0.0, keep_token=None, keep=1, gated=False):
    """One layer, one token: predict -> window update -> insert -> FFN.  ``act`` overrides the
    predicted active list (used to follow another implementation's borderline decisions).
    ``whole_cache`` runs the FFN over every cached row (matrix[:num_used]) instead of only the
    rows of the currently active neurons."""
    logits = predictor_logits(x, A, B, c)
    if act is None:
        act = active_set(logits, theta)
    if keep > 1 and keep_token is None:
        keep_token = keep_tokens(logits, theta, act, keep)
    lists = cache.window_update(act, keep_token, keep)
    cache.insert(lists, bundles, bias_up)
    slots = np.arange(cache.num_used) if whole_cache else lists["active_slots"]
    y = sparse_ffn(cache.matrix, cache.bias, slots, x, b_down, activation, threshold, gated)
    return logits, act, lists, y


def decode_step_gate_predictor(cache, x, gate_matrix, gate_bias, bundles, b_down=None,
                               whole_cache=False, act=None, activation=FATRELU, threshold=0.0):
    """One layer, one token with the resident gate projection as the predictor (Appendix C,
    Llama 2, "alternative approaches"): scores = gate pre-activations, active iff a score
    exceeds the activation's threshold (0 for ReLU), bundles = up | down, and the FFN reuses
    the scores as gate values.  Rows cached but not active now contribute act(gate) = 0."""
    g = gate_scores(x, gate_matrix, gate_bias)
    theta = threshold if activation == FATRELU else 0.0
    if act is None:
        act = active_set(g, theta)
    lists = cache.window_update(act)
    # the per-row scalars still follow the neurons (Section 3.3), though this FFN does not use them
    cache.insert(lists, bundles, gate_bias if gate_bias is not None
                 else np.zeros(cache.d_ff, dtype=np.float16))
    slots = np.arange(cache.num_used) if whole_cache else lists["active_slots"]
    ids = cache.pointers[np.asarray(slots, dtype=np.int64)]
    y = sparse_ffn(cache.matrix, cache.bias, slots, x, b_down, activation, threshold,
                   gate_pre=g[:, ids])
    return g, act, lists, y


# --------------------------------------------------------------------------------------
# Neuron sharding over several devices (not in the paper, which runs on one device: it follows
# from Section 3.3 item 3 -- the FFN output is a sum of one term per cached neuron, in any row
# order -- and from the window rule of Section 3.1 being a per-neuron rule)
# --------------------------------------------------------------------------------------
def neuron_shard_range(d_ff, rank, world):
    """Contiguous id range [lo, hi) of the neurons device ``rank`` of ``world`` owns: equal
    shares of d_ff / world neurons (d_ff must divide evenly)."""
    if world < 1 or not 0 <= rank < world or d_ff % world:
        raise ValueError("d_ff must be a multiple of the number of shards")
    per = d_ff // world
    return rank * per, (rank + 1) * per


def sharded_decode_step(caches, x, A, B, c, theta, bundles, bias_up, b_down=None,
                        whole_cache=False, activation=RELU, threshold=0.0):
    """One layer, one token with the neurons split over len(caches) devices.  Device g owns the
    bundles, predictor columns, offsets and biases of its id range and its own window cache
    (local ids = global id - lo); the input x and the factor A are on every device.  Each
    device runs the ordinary step on its share and produces a partial output; the layer's
    output is the sum of the partials (the one exchange of the step), with the down-projection
    bias added once.  Returns the per-device (logits, act, lists, partial y) and the sum."""
    world = len(caches)
    F = np.asarray(B).shape[1]
    parts = []
    y = None
    for g, cache in enumerate(caches):
        lo, hi = neuron_shard_range(F, g, world)
        part = decode_step(cache, x, A, np.asarray(B)[:, lo:hi], np.asarray(c)[lo:hi], theta,
                           np.asarray(bundles)[lo:hi], np.asarray(bias_up)[lo:hi], None,
                           whole_cache, None, activation, threshold)
        parts.append(part)
        y = part[3] if y is None else y + part[3]
    if b_down is not None:
        y = y + np.asarray(b_down, dtype=np.float64)[None, :]
    return parts, y


# --------------------------------------------------------------------------------------
# The paper's latency / memory accounting (Section 3 intro, Table 1, Appendix C)
# --------------------------------------------------------------------------------------
def io_latency_ms(gigabytes, throughput_gb_per_s):
    """I/O latency = data moved / achieved throughput (Table 1)."""
    return 1000.0 * gigabytes / throughput_gb_per_s


def chunk_bytes(d_model, num_bytes, bundled=True):
    """Bytes per read: d_model * num_bytes for a lone row or column, doubled by bundling
    (Section 3.2)."""
    return (2 if bundled else 1) * d_model * num_bytes


def dram_share_percent(fixed_percents, ffn_percent_of_model, ffn_fraction_resident):
    """Share of the model kept in DRAM = always-resident parts + the cached part of the FFN
    (Appendix C, per-model paragraphs)."""
    return float(sum(fixed_percents) + ffn_fraction_resident * ffn_percent_of_model)


def flash_to_dram_gb(model_gb, ffn_percent_of_model, fraction_of_ffn_per_token):
    """Data loaded per token = model size * FFN share * fraction of FFN neurons needed."""
    return model_gb * ffn_percent_of_model / 100.0 * fraction_of_ffn_per_token


def average_predictor_rank(layer_counts, ranks):
    """Mean predictor rank over the layers when groups of layers use different ranks
    (Appendix B, overhead of predictors: most layers rank 128, the last four rank 1024)."""
    layer_counts = np.asarray(layer_counts, dtype=np.float64)
    return float((layer_counts * np.asarray(ranks, dtype=np.float64)).sum() / layer_counts.sum())


def predictor_weight_fraction(rank, d_model, d_ff, non_embedding_per_layer=None):
    """Predictor parameters r*(d_model + d_ff) relative to a transformer layer's
    4*d^2 (attention) + 2*d*d_ff (FFN) weights (Appendix B, overhead of predictors)."""
    if non_embedding_per_layer is None:
        non_embedding_per_layer = 4 * d_model * d_model + 2 * d_model * d_ff
    return rank * (d_model + d_ff) / non_embedding_per_layer


def kv_cache_fraction(context, d_model, n_layers, model_params):
    """KV cache elements (context * 2 * d_model per layer) over model parameters
    (Appendix C footnote)."""
    return context * 2 * d_model * n_layers / model_params
