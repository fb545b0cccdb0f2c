"""The file-backed bundle store on the host (no GPU): what the reader threads return is the
file's bytes, for aligned and unaligned bundle sizes, cached and uncached reads."""
import os

import numpy as np
import pytest

from paper_2312_11514_b200 import binding as B


def _store_file(tmp_path, n, nbytes, seed=0):
    rng = np.random.default_rng(seed)
    data = rng.integers(0, 256, size=(n, nbytes), dtype=np.uint8)
    path = os.path.join(tmp_path, f"bundles_{nbytes}.bin")
    data.tofile(path)
    return path, data


@pytest.mark.parametrize("nbytes", [4096, 1056, 16384, 18176, 528])
@pytest.mark.parametrize("direct", [True, False])
def test_reader_threads_return_the_files_bundles(tmp_path, nbytes, direct):
    n = 300
    path, data = _store_file(str(tmp_path), n, nbytes)
    store = B.lif_store_open(path, n, nbytes, n_threads=8, direct_io=direct)
    try:
        rng = np.random.default_rng(1)
        for count in (0, 1, 7, 64, 300):
            ids = rng.permutation(n)[:count].astype(np.int32)
            dst = np.full((max(count, 1), nbytes), 0xEE, dtype=np.uint8)
            B.lif_store_read(store, ids, dst)
            np.testing.assert_array_equal(dst[:count], data[ids])
        # the same id twice, the first and the last bundle of the file
        ids = np.array([0, n - 1, 0, n - 1], dtype=np.int32)
        dst = np.zeros((4, nbytes), dtype=np.uint8)
        B.lif_store_read(store, ids, dst)
        np.testing.assert_array_equal(dst, data[ids])
        st = B.lif_store_get_stats(store)
        assert st.n_threads == 8 and st.bytes_requested == (1 + 7 + 64 + 300 + 4) * nbytes
        assert st.bytes_read >= st.bytes_requested and st.reads >= 376
        assert st.direct_io in (0, 1) and (st.direct_io == 0 or direct)
    finally:
        B.lif_store_close(store)


def test_store_rejects_bad_arguments(tmp_path):
    path, data = _store_file(str(tmp_path), 10, 64)
    for bad in (dict(n_bundles=0), dict(bundle_bytes=24), dict(n_threads=0), dict(n_threads=1000),
                dict(n_bundles=11)):                       # 11 bundles do not fit the file
        kw = dict(n_bundles=10, bundle_bytes=64, n_threads=2)
        kw.update(bad)
        with pytest.raises(B.LifError) as e:
            B.lif_store_open(path, kw["n_bundles"], kw["bundle_bytes"], kw["n_threads"], False)
        assert e.value.code == B.LIF_ERR_INVALID_ARG, bad
    with pytest.raises(B.LifError):
        B.lif_store_open(os.path.join(str(tmp_path), "missing.bin"), 10, 64, 2, False)
    store = B.lif_store_open(path, 10, 64, 2, False)
    dst = np.zeros((2, 64), dtype=np.uint8)
    for ids in ([0, 10], [-1, 3]):
        with pytest.raises(B.LifError) as e:
            B.lif_store_read(store, np.array(ids, dtype=np.int32), dst)
        assert e.value.code == B.LIF_ERR_INVALID_ARG
    assert (dst == 0).all()
    B.lif_store_close(store)
    lib = B.lib()
    assert lib.lif_store_close(None) == B.LIF_ERR_INVALID_ARG
    assert lib.lif_decode_step_store(None, None, None, None, None) == B.LIF_ERR_INVALID_ARG
    d = B.make_desc(d_model=256, d_ff=1024, rank=16, window_k=5, capacity=256, staging_rows=100)
    with pytest.raises(B.LifError) as e:                   # a staging buffer smaller than the cache
        B.lif_workspace_bytes(d)
    assert e.value.code == B.LIF_ERR_INVALID_ARG
