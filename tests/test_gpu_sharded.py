"""Neuron sharding on one GPU: the shares of G devices are created as G layers on the same
device (the same calls each device would make on its own share), every share is followed by
its own oracle, and the sum of the partial outputs is compared with the oracle of the unsplit
layer.  The exchange itself (an all-reduce of [n_streams][d_model] fp32 per layer) is covered
on CPU ranks in test_multirank_cpu.py."""
import numpy as np
import pytest
import torch

from oracle import lif_oracle as O
from paper_2312_11514_b200 import binding as B
from paper_2312_11514_b200 import runtime as R
from paper_2312_11514_b200 import workloads as W

import parity_util as P

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bias_down(cfg, n_layers):
    g = torch.Generator(device="cpu").manual_seed(4242)
    return [(torch.randn(cfg.d_model, generator=g) * 0.1).to(torch.float16) for _ in range(n_layers)]


@pytest.mark.parametrize("name,scale,G,n_layers,n_tokens,append_first", [
    ("tiny", {}, 2, 2, 14, 0),
    ("tiny", {}, 4, 2, 14, 1),
    ("opt6p7b", dict(d_model=1024, d_ff=6144, rank=64), 3, 1, 10, 1),
    ("batched8", dict(d_model=512, d_ff=4096, rank=32, n_streams=4), 2, 1, 8, 0),
])
def test_shares_follow_their_oracles_and_sum_to_the_unsplit_layer(name, scale, G, n_layers, n_tokens,
                                                                 append_first):
    cfg = W.CONFIGS[name].scaled(**scale) if scale else W.CONFIGS[name]
    d, F, S = cfg.d_model, cfg.d_ff, cfg.n_streams
    bd = _bias_down(cfg, n_layers)
    stacks = [R.build_stack(cfg, DEV, n_layers=n_layers, shard=(g, G), bias_down=bd,
                            append_first=append_first) for g in range(G)]
    # the oracle's twins: per share (down bias on the first share only) and unsplit
    shares, whole = [], []
    for l in range(n_layers):
        w = W.make_layer(cfg, l, device=DEV)
        row = []
        for g in range(G):
            lo, hi = O.neuron_shard_range(F, g, G)
            gpu = stacks[g][l]
            assert gpu.d_ff == hi - lo
            row.append(P.OracleLayer(W.slice_layer(w, lo, hi), d, hi - lo, gpu.capacity, cfg.window_k,
                                     b_down=bd[l] if g == 0 else None, append_first=append_first))
        shares.append(row)
        whole.append(P.OracleLayer(w, d, F, F, cfg.window_k, b_down=bd[l], append_first=append_first))
    X = W.make_inputs(cfg, device=DEV)
    y = torch.zeros(G, S, d, dtype=torch.float32, device=DEV)
    for t in range(min(n_tokens, cfg.steps)):
        x_np = X[t].cpu().numpy()
        for l in range(n_layers):
            act_all = []
            for g in range(G):
                B.lif_decode_step(stacks[g][l].handle, X[t], y[g])
                torch.cuda.synchronize()
                lists = P.check_decode_step(stacks[g][l], shares[l][g], x_np, y[g])
                lo, _ = O.neuron_shard_range(F, g, G)
                act_all.extend((stacks[g][l].lists()["active_idx"] + lo).tolist())
            y_sum = y.sum(dim=0).cpu().numpy().astype(np.float64)
            # the unsplit oracle, run from the union of the shares' active lists
            ora = whole[l]
            act = np.asarray(act_all, dtype=np.int32)
            P.assert_mask_borderline(act, ora.scores(x_np), ora.theta)
            ls = ora.cache.window_update(act)
            ora.cache.insert(ls, ora.bundles, ora.bias_up)
            ref, _ = P.ffn_reference(ora, ls["active_slots"], x_np)
            P.assert_y_close(y_sum, ref)
            cached = set()
            for g in range(G):
                lo, _ = O.neuron_shard_range(F, g, G)
                st = stacks[g][l].lists()
                cached |= {int(i) + lo for i in st["pointers"][: st["num_used"]]}
            assert cached == ora.cache.cached_ids()
            assert sum(B.lif_get_stats(stacks[g][l].handle).bytes_fetched for g in range(G)) \
                == ora.cache.bytes_fetched
    for st in stacks:
        for layer in st:
            layer.close()



@pytest.mark.parametrize("G,n", [(1, 8), (2, 4096), (5, 4 * 7168 + 4), (16, 300_000)])
def test_peer_sum_adds_the_partials_in_rank_order(G, n):
    # The partials of G devices stand on this one device (a peer's mapped memory is read the
    # same way).  fp32 sums in the stated order are exact to compute on the CPU, so the
    # comparison is bit for bit; in place over the first partial gives the same bits.
    g = torch.Generator(device="cpu").manual_seed(G * 1000 + n)
    parts = [(torch.randn(n, generator=g) * 10 ** float(torch.randint(-3, 3, (1,), generator=g)))
             .to(DEV) for _ in range(G)]
    y = torch.full((n,), float("nan"), device=DEV)
    B.lif_sum_peer_outputs(parts, y)
    torch.cuda.synchronize()
    want = np.zeros(n, dtype=np.float32)
    for p in parts:
        want = (want + p.cpu().numpy()).astype(np.float32)
    np.testing.assert_array_equal(y.cpu().numpy(), want)
    B.lif_sum_peer_outputs(parts, parts[0])
    torch.cuda.synchronize()
    np.testing.assert_array_equal(parts[0].cpu().numpy(), want)


def test_peer_sum_argument_checks():
    y = torch.zeros(16, device=DEV)
    a = torch.zeros(20, device=DEV)
    with pytest.raises(B.LifError):
        B.lif_sum_peer_outputs([a[1:17]], y)                 # misaligned partial
    with pytest.raises(B.LifError):
        B.lif_sum_peer_outputs([a[:16]] * 17, y)             # more than LIF_MAX_PEERS
    with pytest.raises(B.LifError):
        B.lif_sum_peer_outputs([a[:14]], y[:14])             # not a multiple of 4
    assert B.lib().lif_sum_peer_outputs(None, 1, None, 4, None) == B.LIF_ERR_INVALID_ARG
