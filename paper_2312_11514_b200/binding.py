"""ctypes binding of liblif.so.  Argument marshalling only: every function forwards to the C
entry point of the same name (include/lif.h); tensors are passed as raw addresses and
``torch.cuda.Stream.cuda_stream`` handles.  There is no fallback: if the library is missing
or cannot be loaded, importing users get an error."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "liblif.so")

LIF_OK, LIF_ERR_INVALID_ARG, LIF_ERR_ALIGNMENT, LIF_ERR_CAPACITY, LIF_ERR_STATE, LIF_ERR_CUDA, \
    LIF_ERR_TIMEOUT = range(7)
(CNT_N_ACTIVE, CNT_N_EVICT, CNT_N_MOVES, CNT_N_LOAD, CNT_N_HITS, CNT_NUM_USED_BEFORE,
 CNT_NUM_KEPT, CNT_NUM_USED, CNT_STEP, CNT_STATUS, CNT_K_EFF) = range(11)
CNT_LEN = 64
ACT_RELU, ACT_RELU_SQUARED, ACT_FATRELU = range(3)
GATE_NONE, GATE_BUNDLED, GATE_RESIDENT = range(3)

EXPORTS = [
    "lif_status_str", "lif_workspace_bytes", "lif_create_layer", "lif_destroy_layer", "lif_reset",
    "lif_predict", "lif_window_update", "lif_fetch_bundles", "lif_sparse_ffn", "lif_decode_step",
    "lif_decode_token_host", "lif_get_lists", "lif_get_stats", "lif_clear_status",
    "lif_probe_host_read", "lif_probe_device_read", "lif_probe_bulk_ring", "lif_timing_enable", "lif_timing_read",
    "lif_graph_capture", "lif_graph_launch", "lif_graph_launch_host", "lif_graph_destroy",
    "lif_sparse_ffn_static", "lif_sparse_ffn_static_status", "lif_set_tuning", "lif_profile_launch",
    "lif_read_state", "lif_snapshot_bytes", "lif_snapshot", "lif_restore", "lif_sum_peer_outputs",
    "lif_store_open", "lif_store_close", "lif_store_read", "lif_store_get_stats", "lif_decode_step_store",
]
KERNELS = ("predict_z", "predict_scores", "fetch", "ffn_active", "ffn_hits", "ffn_new", "ffn_sum",
           "ffn_cache")
(TUNE_DEPENDENT_LAUNCH, TUNE_SPLIT_FFN, TUNE_FETCH_CTAS, TUNE_FFN_CTAS, TUNE_FFN_STAGES,
 TUNE_BATCHED_COLUMN_PARTS, TUNE_FUSED_PLAN, TUNE_BATCHED_UP_TWO_CTAS, TUNE_FUSED_FETCH_FFN,
 TUNE_WAIT_POLLS, TUNE_EARLY_FETCH) = range(11)
PHASES = ("predict_z", "predict_scores", "window", "moves", "fetch", "ffn", "ffn_sum")
PHASE_LEN = 8


class LayerDesc(C.Structure):
    _fields_ = [
        ("d_model", C.c_int32), ("d_ff", C.c_int32), ("rank", C.c_int32), ("window_k", C.c_int32),
        ("capacity", C.c_int32), ("n_streams", C.c_int32), ("threshold_logit", C.c_float),
        ("ffn_mode", C.c_int32), ("activation", C.c_int32), ("activation_threshold", C.c_float),
        ("budget_rows", C.c_int32), ("spec_keep", C.c_int32), ("gate_mode", C.c_int32),
        ("append_first", C.c_int32), ("staging_rows", C.c_int32), ("dev_gate", C.c_void_p), ("host_bundles", C.c_void_p), ("dev_pred_A", C.c_void_p), ("dev_pred_B", C.c_void_p),
        ("dev_pred_c", C.c_void_p), ("dev_bias_up", C.c_void_p), ("dev_bias_down", C.c_void_p),
        ("dev_cache", C.c_void_p), ("dev_workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
    ]


class Lists(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in (
        "counts", "active_idx", "evict_ids", "move_src", "move_dst", "load_ids", "load_slots",
        "active_slots", "hit_slots", "pointers", "slot_of", "last_active", "bias", "keep_token")]


class Stats(C.Structure):
    _fields_ = [("counts", C.c_int32 * 16), ("bytes_fetched", C.c_uint64),
                ("rows_moved", C.c_uint64), ("rows_active", C.c_uint64),
                ("rows_cached", C.c_uint64), ("status", C.c_int32), ("reserved", C.c_int32)]


class StoreStats(C.Structure):
    _fields_ = [("reads", C.c_uint64), ("bytes_read", C.c_uint64), ("bytes_requested", C.c_uint64),
                ("seconds_reading", C.c_double), ("direct_io", C.c_int32), ("n_threads", C.c_int32)]


class LifError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_str(code)} ({code})")


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    """Load liblif.so (building it first if the sources are newer).  Raises if unavailable."""
    global _lib
    if _lib is not None:
        return _lib
    from . import build as _build
    if _build.needs_build():
        _build.build()
    L = C.CDLL(LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    L.lif_status_str.restype = C.c_char_p
    L.lif_status_str.argtypes = [C.c_int]
    sigs = {
        "lif_workspace_bytes": [C.POINTER(LayerDesc), C.POINTER(sz)],
        "lif_create_layer": [C.POINTER(LayerDesc), C.POINTER(vp)],
        "lif_destroy_layer": [vp],
        "lif_reset": [vp, vp],
        "lif_predict": [vp, vp, vp, vp, vp, vp],
        "lif_window_update": [vp, vp, vp, vp],
        "lif_fetch_bundles": [vp, vp],
        "lif_sparse_ffn": [vp, vp, vp, vp, vp, vp],
        "lif_decode_step": [vp, vp, vp, vp, vp],
        "lif_decode_token_host": [C.POINTER(vp), i32, vp, vp, vp, vp, vp, vp],
        "lif_get_lists": [vp, C.POINTER(Lists)],
        "lif_get_stats": [vp, C.POINTER(Stats)],
        "lif_clear_status": [vp, vp],
        "lif_probe_host_read": [vp, vp, sz, sz, vp],
        "lif_probe_device_read": [vp, sz, vp, i32, i32, vp],
        "lif_probe_bulk_ring": [vp, sz, C.c_uint32, i32, i32, i32, i32, vp, vp, vp],
        "lif_graph_capture": [C.POINTER(vp), i32, vp, vp, vp, vp, C.POINTER(vp)],
        "lif_graph_launch": [vp, vp],
        "lif_graph_launch_host": [vp, vp, vp, vp],
        "lif_graph_destroy": [vp],
        "lif_sparse_ffn_static": [vp, i32, vp, vp, vp, vp, vp, vp, i32, vp],
        "lif_sparse_ffn_static_status": [C.POINTER(C.c_int32), i32],
        "lif_sum_peer_outputs": [C.POINTER(vp), i32, vp, sz, vp],
        "lif_store_open": [C.c_char_p, C.c_int64, C.c_int64, i32, i32, C.POINTER(vp)],
        "lif_store_close": [vp],
        "lif_store_read": [vp, vp, i32, vp],
        "lif_store_get_stats": [vp, C.POINTER(StoreStats)],
        "lif_decode_step_store": [vp, vp, vp, vp, vp],
        "lif_set_tuning": [vp, i32, i32],
        "lif_read_state": [vp, vp, vp, vp, vp],
        "lif_snapshot_bytes": [vp, C.POINTER(sz)],
        "lif_snapshot": [vp, vp, sz],
        "lif_restore": [vp, vp, sz],
        "lif_profile_launch": [vp, i32, vp, vp, vp],
        "lif_timing_enable": [vp, i32],
        "lif_timing_read": [vp, C.POINTER(C.c_float), C.POINTER(i32)],
    }
    for name, args in sigs.items():
        fn = getattr(L, name)
        fn.restype = C.c_int
        fn.argtypes = args
    _lib = L
    return L


def status_str(code: int) -> str:
    return lib().lif_status_str(code).decode()


def _check(code: int, where: str) -> None:
    if code != LIF_OK:
        raise LifError(code, where)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    return t if isinstance(t, int) else t.data_ptr()


def _host_ptr(a) -> Optional[int]:
    """Address of a host array: numpy array or CPU tensor."""
    if a is None:
        return None
    if hasattr(a, "ctypes"):
        return a.ctypes.data
    return a.data_ptr()


def _stream(s) -> Optional[int]:
    if s is None:
        return None
    return s.cuda_stream if hasattr(s, "cuda_stream") else int(s)


def make_desc(*, d_model, d_ff, rank, window_k, capacity, n_streams=1, threshold_logit=0.0,
              ffn_mode=0, activation=0, activation_threshold=0.0, budget_rows=0, spec_keep=0,
              gate_mode=0, gate=None, append_first=0, staging_rows=0, host_bundles=None, pred_A=None, pred_B=None, pred_c=None,
              bias_up=None, bias_down=None, cache=None, workspace=None) -> LayerDesc:
    d = LayerDesc()
    d.d_model, d.d_ff, d.rank, d.window_k, d.capacity = d_model, d_ff, rank, window_k, capacity
    d.n_streams, d.threshold_logit, d.ffn_mode, d.activation = n_streams, threshold_logit, ffn_mode, activation
    d.activation_threshold = activation_threshold
    d.budget_rows = budget_rows
    d.spec_keep = spec_keep
    d.gate_mode, d.dev_gate = gate_mode, _ptr(gate)
    d.append_first = append_first
    d.staging_rows = staging_rows
    d.host_bundles = _ptr(host_bundles)
    d.dev_pred_A, d.dev_pred_B, d.dev_pred_c = _ptr(pred_A), _ptr(pred_B), _ptr(pred_c)
    d.dev_bias_up, d.dev_bias_down = _ptr(bias_up), _ptr(bias_down)
    d.dev_cache, d.dev_workspace = _ptr(cache), _ptr(workspace)
    d.workspace_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    return d


def lif_workspace_bytes(desc: LayerDesc) -> int:
    out = C.c_size_t(0)
    _check(lib().lif_workspace_bytes(C.byref(desc), C.byref(out)), "lif_workspace_bytes")
    return out.value


def lif_create_layer(desc: LayerDesc) -> int:
    out = C.c_void_p(None)
    _check(lib().lif_create_layer(C.byref(desc), C.byref(out)), "lif_create_layer")
    return out.value


def lif_destroy_layer(layer: int) -> None:
    _check(lib().lif_destroy_layer(layer), "lif_destroy_layer")


def lif_reset(layer: int, stream=None) -> None:
    _check(lib().lif_reset(layer, _stream(stream)), "lif_reset")


def lif_predict(layer: int, x, logits, active_idx, n_active, stream=None) -> None:
    _check(lib().lif_predict(layer, _ptr(x), _ptr(logits), _ptr(active_idx), _ptr(n_active),
                             _stream(stream)), "lif_predict")


def lif_window_update(layer: int, active_idx, n_active, stream=None) -> None:
    _check(lib().lif_window_update(layer, _ptr(active_idx), _ptr(n_active), _stream(stream)),
           "lif_window_update")


def lif_fetch_bundles(layer: int, stream=None) -> None:
    _check(lib().lif_fetch_bundles(layer, _stream(stream)), "lif_fetch_bundles")


def lif_sparse_ffn(layer: int, x, slots, n_slots, y, stream=None) -> None:
    _check(lib().lif_sparse_ffn(layer, _ptr(x), _ptr(slots), _ptr(n_slots), _ptr(y),
                                _stream(stream)), "lif_sparse_ffn")


def lif_decode_step(layer: int, x, y, compute_stream=None, fetch_stream=None) -> None:
    _check(lib().lif_decode_step(layer, _ptr(x), _ptr(y), _stream(compute_stream),
                                 _stream(fetch_stream)), "lif_decode_step")


def lif_decode_token_host(layers, host_x, dev_x, dev_y, host_y, compute_stream=None,
                          fetch_stream=None) -> None:
    arr = (C.c_void_p * len(layers))(*layers)
    _check(lib().lif_decode_token_host(arr, len(layers), _ptr(host_x), _ptr(dev_x), _ptr(dev_y),
                                       _ptr(host_y), _stream(compute_stream),
                                       _stream(fetch_stream)), "lif_decode_token_host")


def lif_get_lists(layer: int) -> Lists:
    out = Lists()
    _check(lib().lif_get_lists(layer, C.byref(out)), "lif_get_lists")
    return out


def lif_get_stats(layer: int) -> Stats:
    out = Stats()
    _check(lib().lif_get_stats(layer, C.byref(out)), "lif_get_stats")
    return out


def lif_clear_status(layer: int, stream=None) -> None:
    _check(lib().lif_clear_status(layer, _stream(stream)), "lif_clear_status")


def lif_probe_device_read(dev_src, nbytes: int, dev_sink, ctas_per_sm: int = 2,
                          dependent_launch: bool = True, stream=None) -> None:
    _check(lib().lif_probe_device_read(_ptr(dev_src), nbytes, _ptr(dev_sink), ctas_per_sm,
                                       1 if dependent_launch else 0, _stream(stream)),
           "lif_probe_device_read")


def lif_probe_bulk_ring(dev_src, nbytes: int, chunk_bytes: int, stages: int, refill_group: int,
                        ctas_per_sm: int, threads_every: int, dev_sink, dev_timeouts, stream=None) -> None:
    _check(lib().lif_probe_bulk_ring(_ptr(dev_src), nbytes, chunk_bytes, stages, refill_group,
                                     ctas_per_sm, threads_every, _ptr(dev_sink), _ptr(dev_timeouts),
                                     _stream(stream)), "lif_probe_bulk_ring")


def lif_probe_host_read(host_src, dev_dst, nbytes: int, chunk_bytes: int, stream=None) -> None:
    _check(lib().lif_probe_host_read(_ptr(host_src), _ptr(dev_dst), nbytes, chunk_bytes,
                                     _stream(stream)), "lif_probe_host_read")


def lif_timing_enable(layer: int, n_steps: int) -> None:
    _check(lib().lif_timing_enable(layer, n_steps), "lif_timing_enable")


def lif_timing_read(layer: int):
    """Returns ({phase: summed microseconds}, steps recorded)."""
    us = (C.c_float * PHASE_LEN)()
    n = C.c_int32(0)
    _check(lib().lif_timing_read(layer, us, C.byref(n)), "lif_timing_read")
    return {p: float(us[i]) for i, p in enumerate(PHASES)}, n.value


def lif_graph_capture(layers, dev_x, dev_y, compute_stream, fetch_stream) -> int:
    arr = (C.c_void_p * len(layers))(*layers)
    out = C.c_void_p(None)
    _check(lib().lif_graph_capture(arr, len(layers), _ptr(dev_x), _ptr(dev_y),
                                   _stream(compute_stream), _stream(fetch_stream), C.byref(out)),
           "lif_graph_capture")
    return out.value


def lif_graph_launch(graph: int, stream=None) -> None:
    _check(lib().lif_graph_launch(graph, _stream(stream)), "lif_graph_launch")


def lif_graph_launch_host(graph: int, host_x, host_y, stream=None) -> None:
    _check(lib().lif_graph_launch_host(graph, _ptr(host_x), _ptr(host_y), _stream(stream)),
           "lif_graph_launch_host")


def lif_graph_destroy(graph: int) -> None:
    _check(lib().lif_graph_destroy(graph), "lif_graph_destroy")


def lif_sparse_ffn_static(matrix, n_rows: int, bias, x, slots, n_slots, bias_down, y, d_model: int,
                          stream=None) -> None:
    """Sparse FFN without a layer or workspace: the partial sums use the library's built-in
    2 MiB device array, so nothing is allocated (see include/lif.h for the sharing rules)."""
    _check(lib().lif_sparse_ffn_static(_ptr(matrix), n_rows, _ptr(bias), _ptr(x), _ptr(slots),
                                       _ptr(n_slots), _ptr(bias_down), _ptr(y), d_model,
                                       _stream(stream)), "lif_sparse_ffn_static")


def lif_sparse_ffn_static_status(clear: bool = True) -> int:
    """Synchronises the device and returns the sticky status word of lif_sparse_ffn_static on
    the current device (a LIF_* code), resetting it when ``clear``."""
    out = C.c_int32(-1)
    _check(lib().lif_sparse_ffn_static_status(C.byref(out), 1 if clear else 0),
           "lif_sparse_ffn_static_status")
    return int(out.value)


def lif_store_open(path: str, n_bundles: int, bundle_bytes: int, n_threads: int = 32,
                   direct_io: bool = True) -> int:
    out = C.c_void_p(None)
    _check(lib().lif_store_open(path.encode(), n_bundles, bundle_bytes, n_threads,
                                1 if direct_io else 0, C.byref(out)), "lif_store_open")
    return out.value


def lif_store_close(store: int) -> None:
    _check(lib().lif_store_close(store), "lif_store_close")


def lif_store_read(store: int, ids, dst) -> None:
    """Bundles ``ids`` (int32 numpy array or CPU tensor) into ``dst`` (host numpy array or CPU
    tensor of len(ids) * bundle_bytes bytes)."""
    _check(lib().lif_store_read(store, _host_ptr(ids), len(ids), _host_ptr(dst)), "lif_store_read")


def lif_store_get_stats(store: int) -> StoreStats:
    out = StoreStats()
    _check(lib().lif_store_get_stats(store, C.byref(out)), "lif_store_get_stats")
    return out


def lif_decode_step_store(layer: int, store: int, x, y, stream=None) -> None:
    _check(lib().lif_decode_step_store(layer, store, _ptr(x), _ptr(y), _stream(stream)),
           "lif_decode_step_store")


def lif_sum_peer_outputs(partials, y, stream=None) -> None:
    """y = partials[0] + partials[1] + ... (fp32 tensors of equal size, this device's or mapped
    peers'; integers are taken as device addresses); see include/lif.h."""
    ptrs = (C.c_void_p * len(partials))(*[p if isinstance(p, int) else _ptr(p) for p in partials])
    _check(lib().lif_sum_peer_outputs(ptrs, len(partials), _ptr(y), y.numel(), _stream(stream)),
           "lif_sum_peer_outputs")


def lif_set_tuning(layer: int, key: int, value: int) -> None:
    _check(lib().lif_set_tuning(layer, key, value), "lif_set_tuning")


def lif_profile_launch(layer: int, kernel: int, x, y, stream=None) -> None:
    _check(lib().lif_profile_launch(layer, kernel, _ptr(x), _ptr(y), _stream(stream)),
           "lif_profile_launch")


def lif_read_state(layer: int, pointers=None, slot_of=None, last_active=None, num_used=None) -> None:
    """Arguments are host int32 numpy arrays (or None)."""
    ptr = lambda a: None if a is None else a.ctypes.data
    _check(lib().lif_read_state(layer, ptr(pointers), ptr(slot_of), ptr(last_active), ptr(num_used)),
           "lif_read_state")


def lif_snapshot(layer: int) -> bytes:
    n = C.c_size_t(0)
    _check(lib().lif_snapshot_bytes(layer, C.byref(n)), "lif_snapshot_bytes")
    buf = C.create_string_buffer(n.value)
    _check(lib().lif_snapshot(layer, C.cast(buf, C.c_void_p), n.value), "lif_snapshot")
    return buf.raw


def lif_restore(layer: int, snapshot: bytes) -> None:
    buf = C.create_string_buffer(snapshot, len(snapshot))
    _check(lib().lif_restore(layer, C.cast(buf, C.c_void_p), len(snapshot)), "lif_restore")
