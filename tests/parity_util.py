"""Shared helpers of the GPU parity tests: tolerances and the teacher-forced comparison of the
CUDA path (through the C ABI) with the CPU oracle, stage by stage."""
import numpy as np
import torch

from oracle import lif_oracle as O
from paper_2312_11514_b200 import binding as B
from paper_2312_11514_b200 import runtime as R
from paper_2312_11514_b200 import workloads as W

REL = 2e-3          # max relative error on FFN outputs and predictor scores (fp16 storage, fp32 accumulate)
BORDER = 1e-3       # mask disagreement is allowed only where |score - theta| < BORDER
LIST_KEYS = ("evict_ids", "move_src", "move_dst", "load_ids", "load_slots", "active_slots", "hit_slots")


def assert_logits_close(got, ref):
    tol = REL * np.maximum(np.abs(ref), 1.0)
    bad = np.abs(got - ref) > tol
    assert not bad.any(), f"{bad.sum()} scores off, worst {np.abs(got - ref).max():.3e}"


def assert_mask_borderline(act_gpu, ref_logits, theta):
    """The GPU's active list may differ from the oracle's only on neurons whose oracle score
    is within BORDER of the threshold."""
    ref_act = O.active_set(ref_logits, theta)
    diff = np.setxor1d(act_gpu, ref_act)
    if diff.size:
        margin = np.abs(ref_logits[:, diff] - theta).min(axis=0)
        assert (margin < BORDER).all(), f"mask differs away from the threshold: {diff[margin >= BORDER]}"
    assert (np.diff(act_gpu) > 0).all()
    return diff.size


def assert_y_close(got, ref, flips=()):
    """``flips``: (stream, delta[d]) pairs, one per FATReLU decision that sits within rounding of
    its threshold: the activation jumps there, so either side of it is a correct result and a
    stream's row of ``got`` may match ``ref`` with any subset of that stream's deltas added."""
    worst = 0.0
    for s_ in range(ref.shape[0]):
        mine = [delta for (t_, delta) in flips if t_ == s_]
        assert len(mine) <= 14, "too many borderline activations in one stream to enumerate"
        best = None
        for subset in range(1 << len(mine)):
            r = ref[s_].copy()
            for j, delta in enumerate(mine):
                if subset >> j & 1:
                    r = r + delta
            tol = REL * np.maximum(np.abs(r), np.sqrt(np.mean(r * r))) + 1e-30
            ratio = (np.abs(got[s_] - r) / tol).max()
            best = ratio if best is None else min(best, ratio)
            if ratio <= 1.0:
                break
        worst = max(worst, best)
    assert worst <= 1.0, f"outputs off, worst ratio {worst:.3f}"


# |pre-activation - FATReLU threshold| below this: the decision may differ (fp32 accumulation of
# up to 8192 fp16 products of O(1) size is off by about 1e-6)
ACT_BORDER = 2e-5


def ffn_reference(ora, slots, x_np, gate_pre=None):
    """Oracle FFN over ``slots`` plus the flips (see assert_y_close) of borderline FATReLU
    decisions.  ``gate_pre`` [S][len(slots)]: resident-gate mode."""
    gated = ora.gate_mode == 1
    ref = O.sparse_ffn(ora.cache.matrix, ora.cache.bias, slots, x_np, ora.b_down, ora.activation,
                       ora.act_threshold, gated=gated, gate_pre=gate_pre)
    flips = []
    if ora.activation == O.FATRELU and ora.act_threshold > 0 and len(slots):
        d = x_np.shape[1]
        rows = ora.cache.matrix[np.asarray(slots, dtype=np.int64)].astype(np.float64)
        x = x_np.astype(np.float64)
        pre = (np.asarray(gate_pre, dtype=np.float64) if gate_pre is not None
               else x @ rows[:, :d].T + ora.cache.bias[slots].astype(np.float64)[None, :])
        mult = np.ones_like(pre) if ora.gate_mode == 0 else x @ rows[:, -2 * d:-d].T
        for s_, q in zip(*np.nonzero(np.abs(pre - ora.act_threshold) < ACT_BORDER)):
            sign = -1.0 if pre[s_, q] > ora.act_threshold else 1.0
            flips.append((s_, sign * pre[s_, q] * mult[s_, q] * rows[q, -d:]))
    return ref, flips


class OracleLayer:
    """Oracle-side twin of one layer, fed with the same tensors."""

    def __init__(self, w, d_model, d_ff, capacity, window_k, theta=0.0, b_down=None,
                 activation=0, act_threshold=0.0, budget_rows=0, gate_mode=0, append_first=False):
        self.activation, self.act_threshold, self.gate_mode = activation, act_threshold, gate_mode
        self.gate = w["gate"].cpu().numpy() if gate_mode == 2 else None
        self.A = w["A"].cpu().numpy().astype(np.float64)
        self.B = w["B"].cpu().numpy().astype(np.float64)
        self.c = w["c"].cpu().numpy().astype(np.float64)
        self.bundles = w["bundles"].cpu().numpy()
        self.bias_up = w["bias_up"].cpu().numpy()
        self.b_down = None if b_down is None else b_down.cpu().numpy()
        self.theta = theta
        if gate_mode == 2:        # the gate is the predictor: active iff it passes the activation
            self.theta = act_threshold if activation == O.FATRELU else 0.0
        self.cache = O.NeuronCache(d_model, d_ff, capacity, window_k, budget_rows,
                                   n_vec=3 if gate_mode == 1 else 2, append_first=bool(append_first))

    def scores(self, x_np):
        """The predictor's scores: low-rank, or the resident gate's pre-activations."""
        if self.gate_mode == 2:
            return O.gate_scores(x_np, self.gate, self.bias_up)
        return O.predictor_logits(x_np, self.A, self.B, self.c)


def make_layer_pair(cfg, layer_idx, *, capacity=None, theta=0.0, ffn_mode=0, b_down=False,
                    activation=0, act_threshold=0.0, budget_rows=0, spec_keep=0, gate_mode=0,
                    append_first=0, store_file=None, device="cuda:0"):
    """``store_file``: write the bundles to this file and give the layer a staging buffer of
    ``capacity`` rows instead of the whole store (it then steps through lif_decode_step_store)."""
    n_vec = 3 if gate_mode == 1 else 2
    store = R.pinned_store(cfg.d_ff, cfg.d_model, n_vec)
    w = W.make_layer(cfg, layer_idx, device=device, bundles_out=store, gate_mode=gate_mode,
                     act_threshold=act_threshold)
    cap = capacity or W.window_capacity(cfg, w["p"])
    staging_rows = 0
    if store_file is not None:
        store.numpy().tofile(store_file)
        staging_rows = cap
        store = torch.zeros(cap, n_vec * cfg.d_model, dtype=torch.float16).pin_memory()
    bd = None
    if b_down:
        g = torch.Generator(device="cpu").manual_seed(77 + layer_idx)
        bd = (torch.randn(cfg.d_model, generator=g) * 0.1).to(torch.float16).to(device)
    dev = lambda t: t.to(device).contiguous()
    gpu = R.Layer(d_model=cfg.d_model, d_ff=cfg.d_ff, rank=cfg.rank, window_k=cfg.window_k,
                  capacity=cap, host_bundles=store, pred_A=dev(w["A"]), pred_B=dev(w["B"]),
                  pred_c=dev(w["c"]), bias_up=dev(w["bias_up"]), bias_down=bd,
                  n_streams=cfg.n_streams, threshold_logit=theta, ffn_mode=ffn_mode,
                  activation=activation, activation_threshold=act_threshold, budget_rows=budget_rows,
                  spec_keep=spec_keep, gate_mode=gate_mode,
                  gate=dev(w["gate"]) if gate_mode == 2 else None, append_first=append_first,
                  staging_rows=staging_rows, device=device)
    ora = OracleLayer(w, cfg.d_model, cfg.d_ff, cap, cfg.window_k, theta, bd, activation, act_threshold,
                      budget_rows, gate_mode, append_first)
    return gpu, ora


def compare_lists_and_state(gpu, ora, ref_lists):
    g = gpu.lists()
    assert g["status"] == B.LIF_OK
    for key in LIST_KEYS:
        np.testing.assert_array_equal(g[key], ref_lists[key], err_msg=key)
    for key in ("num_used_before", "num_kept", "num_used", "k_eff"):
        assert g[key] == ref_lists[key], key
    c = ora.cache
    assert g["step"] == c.t
    np.testing.assert_array_equal(g["pointers"], c.pointers)
    np.testing.assert_array_equal(g["slot_of"], c.slot_of)
    np.testing.assert_array_equal(g["last_active"], c.last_active)
    return g


def compare_cache_rows(gpu, ora):
    n = ora.cache.num_used
    rows = gpu.cache[:n].cpu().numpy()
    assert np.array_equal(rows.view(np.uint16), ora.cache.matrix[:n].view(np.uint16))
    bias = gpu.lists()["bias"][:n]
    assert np.array_equal(bias.view(np.uint16), ora.cache.bias[:n].view(np.uint16))


def keep_tokens_checked(gpu, act_gpu, ref_logits, theta):
    """Speculative mode: the GPU's per-neuron last kept token, checked against the oracle's
    scores (it may differ only where a score of a kept token is within BORDER of the
    threshold); the oracle then continues from the GPU's values."""
    keep = gpu.spec_keep
    torch.cuda.synchronize()
    kt_gpu = gpu._view("keep_token", gpu.d_ff, torch.int8).cpu().numpy().astype(np.int64)[act_gpu]
    kt_ref = O.keep_tokens(ref_logits, theta, act_gpu, keep)
    diff = np.nonzero(kt_gpu != kt_ref)[0]
    if diff.size:
        margin = np.abs(ref_logits[:keep][:, act_gpu[diff]] - theta).min(axis=0)
        assert (margin < BORDER).all(), "kept-token index differs away from the threshold"
    assert ((kt_gpu >= -1) & (kt_gpu < keep)).all()
    return kt_gpu


def make_bufs(gpu, device="cuda:0"):
    S, F, d = gpu.n_streams, gpu.d_ff, gpu.d_model
    return dict(logits=torch.empty(S, F, dtype=torch.float32, device=device),
                act=torch.empty(F, dtype=torch.int32, device=device),
                n_act=torch.zeros(1, dtype=torch.int32, device=device),
                y=torch.empty(S, d, dtype=torch.float32, device=device))


def staged_step(gpu, ora, x_dev, bufs, whole_cache=False):
    """One token through the four staged entry points, each compared with the oracle run from
    the GPU's own active list (so borderline predictor decisions do not cascade)."""
    F = gpu.d_ff
    logits, act, n_act, y = bufs["logits"], bufs["act"], bufs["n_act"], bufs["y"]
    B.lif_predict(gpu.handle, x_dev, logits, act, n_act)
    torch.cuda.synchronize()
    x_np = x_dev.cpu().numpy()
    ref_logits = ora.scores(x_np)
    assert_logits_close(logits.cpu().numpy().astype(np.float64), ref_logits)
    na = int(n_act.item())
    act_gpu = act[:na].cpu().numpy()
    n_border = assert_mask_borderline(act_gpu, ref_logits, ora.theta)

    kt, keep = None, 1
    if gpu.spec_keep > 0:
        kt, keep = keep_tokens_checked(gpu, act_gpu, ref_logits, ora.theta), gpu.spec_keep
    B.lif_window_update(gpu.handle, act, n_act)
    ref_lists = ora.cache.window_update(act_gpu, kt, keep)
    g = compare_lists_and_state(gpu, ora, ref_lists)
    np.testing.assert_array_equal(g["active_idx"], act_gpu)

    B.lif_fetch_bundles(gpu.handle)
    ora.cache.insert(ref_lists, ora.bundles, ora.bias_up)
    compare_cache_rows(gpu, ora)

    if whole_cache:
        B.lif_sparse_ffn(gpu.handle, x_dev, None, gpu.counts[B.CNT_NUM_USED:], y)
        slots = np.arange(ora.cache.num_used)
    else:
        B.lif_sparse_ffn(gpu.handle, x_dev, gpu._view("active_slots", F),
                         gpu.counts[B.CNT_N_ACTIVE:], y)
        slots = ref_lists["active_slots"]
    torch.cuda.synchronize()
    gate_pre = None
    if ora.gate_mode == 2:
        gate_pre = ref_logits[:, ora.cache.pointers[np.asarray(slots, dtype=np.int64)]]
    ref_y, flips = ffn_reference(ora, slots, x_np, gate_pre)
    assert_y_close(y.cpu().numpy().astype(np.float64), ref_y, flips)
    return dict(n_active=na, n_load=len(ref_lists["load_ids"]), n_evict=len(ref_lists["evict_ids"]),
                n_border=n_border, k_eff=ref_lists["k_eff"], num_used=ref_lists["num_used"])


def check_decode_step(gpu, ora, x_np, y):
    """After one lif_decode_step of ``gpu`` on ``x_np``: the active list may differ from the
    oracle's only at borderline scores; from that list on, the oracle reproduces lists, window
    state and (within tolerance) the output ``y`` [S][d] (a device tensor, read here after the
    device has been synchronised, or an array the caller read after synchronising).  Returns
    the step's lists."""
    g = gpu.lists()                    # synchronises the device
    y_np = y.cpu().numpy().astype(np.float64) if isinstance(y, torch.Tensor) else y
    assert g["status"] == B.LIF_OK, f"device status {g['status']}"
    scores = ora.scores(x_np)
    assert_mask_borderline(g["active_idx"], scores, ora.theta)
    lists = ora.cache.window_update(g["active_idx"])
    ora.cache.insert(lists, ora.bundles, ora.bias_up)
    compare_lists_and_state(gpu, ora, lists)
    slots = lists["active_slots"]
    gate_pre = scores[:, g["active_idx"]] if ora.gate_mode == 2 else None
    ref_y, flips = ffn_reference(ora, slots, x_np, gate_pre)
    assert_y_close(y_np, ref_y, flips)
    return lists
