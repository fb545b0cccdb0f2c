"""The bundle store in a file (the paper's storage tier: reader threads, one read per bundle,
uncached where the file system allows) feeding the same layer: lists, window state, cache rows
and outputs must be what the oracle computes, exactly as with the pinned-memory store."""
import numpy as np
import pytest
import torch

from paper_2312_11514_b200 import binding as B
from paper_2312_11514_b200 import workloads as W

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("d,F,S,append_first,direct", [
    (264, 1000, 1, 0, True),      # 1056-byte bundles: read through an aligned window
    (1024, 2048, 1, 1, True),     # 4096-byte bundles: read straight into the staging buffer
    (512, 1536, 3, 1, False),     # three streams (tensor-core FFN), reads through the page cache
])
def test_decode_steps_from_a_file_store_follow_the_oracle(tmp_path, d, F, S, append_first, direct):
    cfg = W.LifConfig("file", 1, d, F, 16, 3, S, 10, 0.08, 1.0, 0.8, 0.6, 44)
    path = str(tmp_path / "bundles.bin")
    gpu, ora = P.make_layer_pair(cfg, 0, b_down=True, append_first=append_first, store_file=path)
    store = B.lif_store_open(path, F, 4 * d, n_threads=8, direct_io=direct)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(S, d, dtype=torch.float32, device=DEV)
    st = torch.cuda.Stream()
    torch.cuda.synchronize()
    loaded = 0
    for t in range(cfg.steps):
        B.lif_decode_step_store(gpu.handle, store, X[t], y, st)
        lists = P.check_decode_step(gpu, ora, X[t].cpu().numpy(), y)
        P.compare_cache_rows(gpu, ora)             # every cached row is the file's bundle
        loaded += len(lists["load_ids"])
    stats = B.lif_store_get_stats(store)
    assert stats.bytes_requested == loaded * 4 * d == ora.cache.bytes_fetched
    assert stats.bytes_read >= stats.bytes_requested and stats.n_threads == 8
    if not direct:
        assert stats.direct_io == 0
    # the calls that would read host_bundles by neuron id refuse a staging buffer
    for call in (lambda: B.lif_decode_step(gpu.handle, X[0], y), lambda: B.lif_fetch_bundles(gpu.handle),
                 lambda: B.lif_restore(gpu.handle, B.lif_snapshot(gpu.handle))):
        with pytest.raises(B.LifError) as e:
            call()
        assert e.value.code == B.LIF_ERR_STATE
    B.lif_store_close(store)
    gpu.close()


def test_file_store_of_another_shape_is_refused(tmp_path):
    cfg = W.LifConfig("file", 1, 256, 512, 16, 3, 1, 4, 0.08, 1.0, 0.8, 0.6, 45)
    path = str(tmp_path / "bundles.bin")
    gpu, ora = P.make_layer_pair(cfg, 0, store_file=path)
    X = W.make_inputs(cfg, device=DEV)
    y = torch.empty(1, 256, dtype=torch.float32, device=DEV)
    wrong = B.lif_store_open(path, 256, 4 * 256, n_threads=2, direct_io=False)   # half the neurons
    with pytest.raises(B.LifError) as e:
        B.lif_decode_step_store(gpu.handle, wrong, X[0], y)
    assert e.value.code == B.LIF_ERR_INVALID_ARG
    B.lif_store_close(wrong)
    # a layer over a whole pinned store cannot step from a file either way round: it has no
    # staging buffer declared, and its host_bundles must not be overwritten
    full, _ = P.make_layer_pair(cfg, 0)
    ok = B.lif_store_open(path, 512, 4 * 256, n_threads=2, direct_io=False)
    with pytest.raises(B.LifError) as e:
        B.lif_decode_step_store(full.handle, ok, X[0], y)
    assert e.value.code == B.LIF_ERR_STATE
    B.lif_store_close(ok)
    full.close()
    gpu.close()
