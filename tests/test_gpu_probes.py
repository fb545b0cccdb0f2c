"""The profiling aids of lif_profile.h that bench.py --floors is built on: they run, touch only
what they are given, and refuse sizes they cannot handle."""
import pytest
import torch

from paper_2312_11514_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_device_read_and_ring_probes_run_to_completion():
    n = 8 << 20
    src = torch.arange(n // 4, dtype=torch.int32, device=DEV)
    guard_before = src.clone()
    sink = torch.zeros(4, dtype=torch.int32, device=DEV)
    tmo = torch.zeros(1, dtype=torch.int32, device=DEV)
    st = torch.cuda.Stream()
    torch.cuda.synchronize()
    for ctas in (1, 4):
        for pdl in (True, False):
            B.lif_probe_device_read(src, n, sink, ctas, pdl, st)
    for chunk, stages, group, ctas, every in ((3584, 48, 16, 1, 0), (14336, 16, 8, 1, 0), (7168, 14, 7, 2, 0),
                                              (7168, 32, 16, 1, 2), (4096, 8, 4, 4, 1), (2048, 6, 6, 1, 0)):
        B.lif_probe_bulk_ring(src, n, chunk, stages, group, ctas, every, sink, tmo, st)
    torch.cuda.synchronize()
    assert int(tmo.item()) == 0                      # no bounded wait ran out
    assert torch.equal(src, guard_before) and int(sink.abs().sum()) == 0
    # an odd tail: bytes that are not a multiple of CTAs x chunk are simply not read
    B.lif_probe_bulk_ring(src, n - 4096, 7168, 32, 16, 1, 0, sink, tmo, st)
    torch.cuda.synchronize()
    assert int(tmo.item()) == 0


def test_probes_refuse_bad_arguments():
    src = torch.zeros(1 << 20, dtype=torch.uint8, device=DEV)
    sink = torch.zeros(16, dtype=torch.uint8, device=DEV)
    tmo = torch.zeros(1, dtype=torch.int32, device=DEV)
    for args in ((src, 1 << 20, 100, 8, 4, 1, 0), (src, 1 << 20, 4096, 8, 3, 1, 0), (src, 1 << 20, 4096, 0, 1, 1, 0),
                 (src, 1 << 20, 4096, 8, 4, 9, 0), (src, 1 << 20, 65536, 8, 4, 1, 0),   # ring beyond shared memory
                 (src, 4096, 4096, 8, 4, 1, 0)):                                        # less than a chunk per CTA
        with pytest.raises(B.LifError) as e:
            B.lif_probe_bulk_ring(*args, sink, tmo)
        assert e.value.code == B.LIF_ERR_INVALID_ARG, args
    with pytest.raises(B.LifError) as e:
        B.lif_probe_bulk_ring(src[8:], 1 << 19, 4096, 8, 4, 1, 0, sink, tmo)
    assert e.value.code == B.LIF_ERR_ALIGNMENT
    for args in ((src, 0, sink, 2, True), (src, 100, sink, 2, True), (src, 4096, sink, 0, True), (src, 4096, sink, 9, True)):
        with pytest.raises(B.LifError) as e:
            B.lif_probe_device_read(*args)
        assert e.value.code == B.LIF_ERR_INVALID_ARG, args
