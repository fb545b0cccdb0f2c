"""Host-only checks of the C ABI: the library builds, loads, exports every symbol the header
declares, and rejects bad descriptions before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2312_11514_b200 import binding as B

INCLUDE = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include")


def _declared():
    names = set()
    for header in sorted(os.listdir(INCLUDE)):
        text = open(os.path.join(INCLUDE, header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(lif_[a-z_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    lib = B.lib()
    names = _declared()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(B.EXPORTS) == names


def test_status_strings():
    assert B.status_str(B.LIF_OK) == "ok"
    assert "capacity" in B.status_str(B.LIF_ERR_CAPACITY)
    assert len({B.status_str(i) for i in range(7)}) == 7


def _shape(**kw):
    base = dict(d_model=256, d_ff=1024, rank=16, window_k=5, capacity=256)
    base.update(kw)
    return B.make_desc(**base)


def test_workspace_bytes_and_shape_validation():
    n = B.lif_workspace_bytes(_shape())
    assert n > 0 and n % 256 == 0
    assert B.lif_workspace_bytes(_shape(d_ff=2048, capacity=512)) > n
    for bad in (dict(d_model=260), dict(d_model=0), dict(d_model=16384), dict(d_ff=1001), dict(rank=12),
                dict(rank=4096), dict(window_k=0), dict(capacity=0), dict(capacity=2048),
                dict(n_streams=0), dict(n_streams=9), dict(ffn_mode=2), dict(activation=3), dict(activation=-1),
                dict(activation=2, activation_threshold=-0.5), dict(activation=2, activation_threshold=float("nan")),
                dict(threshold_logit=float("nan"))):
        with pytest.raises(B.LifError) as e:
            B.lif_workspace_bytes(_shape(**bad))
        assert e.value.code == B.LIF_ERR_INVALID_ARG, bad


def test_create_layer_rejects_null_and_misaligned_pointers_on_the_host():
    d = _shape()
    with pytest.raises(B.LifError) as e:          # every pointer NULL
        B.lif_create_layer(d)
    assert e.value.code == B.LIF_ERR_INVALID_ARG
    for f in ("host_bundles", "dev_pred_A", "dev_pred_B", "dev_pred_c", "dev_bias_up", "dev_cache",
              "dev_workspace"):
        setattr(d, f, 0x10000)
    d.workspace_bytes = 1 << 30
    d.dev_cache = 0x10008                          # not 16-byte aligned
    with pytest.raises(B.LifError) as e:
        B.lif_create_layer(d)
    assert e.value.code == B.LIF_ERR_ALIGNMENT
    d.dev_cache = 0x10000
    d.workspace_bytes = 16                         # too small
    with pytest.raises(B.LifError) as e:
        B.lif_create_layer(d)
    assert e.value.code == B.LIF_ERR_INVALID_ARG
    out = C.c_void_p(123)
    assert B.lib().lif_create_layer(C.byref(d), None) == B.LIF_ERR_INVALID_ARG
    assert B.lib().lif_destroy_layer(None) == B.LIF_ERR_INVALID_ARG
    assert B.lib().lif_decode_step(None, None, None, None, None) == B.LIF_ERR_INVALID_ARG
    assert B.lib().lif_probe_host_read(None, None, 0, 0, None) == B.LIF_ERR_INVALID_ARG


def test_new_fields_are_validated_on_the_host():
    ok = dict(n_streams=5, spec_keep=2)
    assert B.lif_workspace_bytes(_shape(**ok)) > B.lif_workspace_bytes(_shape(n_streams=5))   # keep_token array
    assert B.lif_workspace_bytes(_shape(budget_rows=128)) > 0
    for bad in (dict(n_streams=4, spec_keep=5), dict(spec_keep=-1), dict(budget_rows=-3),
                dict(budget_rows=512), dict(n_streams=4, spec_keep=2, budget_rows=100),
                dict(window_k=40, budget_rows=100)):
        with pytest.raises(B.LifError) as e:
            B.lif_workspace_bytes(_shape(**bad))
        assert e.value.code == B.LIF_ERR_INVALID_ARG, bad


def test_graph_and_profiling_calls_reject_null_handles():
    lib = B.lib()
    out = C.c_void_p(None)
    assert lib.lif_graph_capture(None, 0, None, None, None, None, C.byref(out)) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_graph_capture(None, 0, None, None, None, None, None) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_graph_launch(None, None) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_graph_launch_host(None, None, None, None) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_graph_destroy(None) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_profile_launch(None, 0, None, None, None) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_set_tuning(None, 0, 0) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_timing_enable(None, 1) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_sparse_ffn_static(None, 1, None, None, None, None, None, None, 256, None) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_sparse_ffn_static_status(None, 0) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_sum_peer_outputs(None, 2, None, 16, None) == B.LIF_ERR_INVALID_ARG


def _enumerators():
    """Every `NAME = integer` enumerator of the headers."""
    values = {}
    for header in sorted(os.listdir(INCLUDE)):
        text = open(os.path.join(INCLUDE, header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        for name, value in re.findall(r"\b(LIF_[A-Z0-9_]+)\s*=\s*(-?\d+)", text):
            values[name] = int(value)
    return values


def test_binding_constants_equal_the_headers_enumerators():
    enums = _enumerators()
    assert len(enums) > 40
    checked = 0
    for name, value in enums.items():
        short = name[4:]                              # the binding drops the LIF_ prefix ...
        for candidate in (name, short):               # ... except for the status codes
            if hasattr(B, candidate):
                assert getattr(B, candidate) == value, name
                checked += 1
                break
    assert checked > 30
    # tuples indexed by enumerator value
    for i, kernel in enumerate(B.KERNELS):
        assert enums["LIF_KERNEL_" + kernel.upper()] == i
    assert enums["LIF_CNT_LEN"] == B.CNT_LEN
