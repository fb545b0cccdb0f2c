"""Device-memory plumbing around the C ABI: allocates the buffers a layer needs with torch
(pinned bundle store, window cache, workspace), creates the layer, and exposes the lists
inside the workspace as tensor views.  No arithmetic of the method lives here."""
from __future__ import annotations

from typing import Dict, List, Optional

import torch

from . import binding as B


class Layer:
    """One FFN layer: owns its torch buffers and the `lif_layer` handle."""

    def __init__(self, *, d_model: int, d_ff: int, rank: int, window_k: int, capacity: int,
                 host_bundles: torch.Tensor, bias_up: torch.Tensor,
                 pred_A: Optional[torch.Tensor] = None, pred_B: Optional[torch.Tensor] = None,
                 pred_c: Optional[torch.Tensor] = None,
                 bias_down: Optional[torch.Tensor] = None, n_streams: int = 1,
                 threshold_logit: float = 0.0, ffn_mode: int = 0, activation: int = 0,
                 activation_threshold: float = 0.0, budget_rows: int = 0, spec_keep: int = 0,
                 gate_mode: int = 0, gate: Optional[torch.Tensor] = None, append_first: int = 0,
                 staging_rows: int = 0, device="cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2312_11514_b200 needs a CUDA device; there is no CPU path")
        self.device = torch.device(device)
        assert host_bundles.is_pinned() and host_bundles.dtype == torch.float16
        n_vec = 3 if gate_mode == B.GATE_BUNDLED else 2      # d_model-vectors per bundle
        # staging_rows > 0: the bundles live in a file and host_bundles is the staging buffer
        assert host_bundles.shape == (staging_rows or d_ff, n_vec * d_model) and host_bundles.is_contiguous()
        assert gate is None or (gate.shape == (d_ff, d_model) and gate.dtype == torch.float16
                                and gate.is_contiguous())
        self.d_model, self.d_ff, self.rank, self.capacity = d_model, d_ff, rank, capacity
        self.n_streams = n_streams
        self.keep = dict(host_bundles=host_bundles, pred_A=pred_A, pred_B=pred_B, pred_c=pred_c,
                         bias_up=bias_up, bias_down=bias_down, gate=gate)
        # One guard row past the cache and a guard block past the workspace, filled with a bit
        # pattern no kernel writes: `guards_intact()` tells whether anything ran past the end.
        self._cache_all = torch.zeros(capacity + 1, n_vec * d_model, dtype=torch.float16, device=self.device)
        self._cache_all[capacity].view(torch.int16).fill_(self._GUARD)
        self.cache = self._cache_all[:capacity]
        shape = dict(d_model=d_model, d_ff=d_ff, rank=rank, window_k=window_k, capacity=capacity,
                     n_streams=n_streams, threshold_logit=threshold_logit, ffn_mode=ffn_mode,
                     activation=activation, activation_threshold=activation_threshold,
                     budget_rows=budget_rows, spec_keep=spec_keep, gate_mode=gate_mode,
                     append_first=append_first, staging_rows=staging_rows)
        self.spec_keep, self.gate_mode = spec_keep, gate_mode
        nbytes = B.lif_workspace_bytes(B.make_desc(**shape))
        self._workspace_all = torch.zeros(nbytes + 256, dtype=torch.uint8, device=self.device)
        self._workspace_all[nbytes:].fill_(self._GUARD & 0xFF)
        self.workspace = self._workspace_all[:nbytes]
        with torch.cuda.device(self.device):
            self.handle = B.lif_create_layer(B.make_desc(
                **shape, host_bundles=host_bundles, pred_A=pred_A, pred_B=pred_B, pred_c=pred_c,
                bias_up=bias_up, bias_down=bias_down, gate=gate, cache=self.cache,
                workspace=self.workspace))
            torch.cuda.synchronize()   # the reset ran on the default stream
        self._lists = B.lif_get_lists(self.handle)
        self.counts = self._view("counts", B.CNT_LEN)

    _GUARD = 0x7B7B

    def guards_intact(self) -> bool:
        """True while the row after the cache and the block after the workspace still hold the
        pattern they were created with (synchronises)."""
        torch.cuda.synchronize(self.device)
        row_ok = bool((self._cache_all[self.capacity].view(torch.int16) == self._GUARD).all())
        ws_ok = bool((self._workspace_all[self.workspace.numel():] == (self._GUARD & 0xFF)).all())
        return row_ok and ws_ok

    def _view(self, name: str, n: int, dtype=torch.int32) -> torch.Tensor:
        off = getattr(self._lists, name) - self.workspace.data_ptr()
        size = n * torch.empty((), dtype=dtype).element_size()
        return self.workspace[off:off + size].view(dtype)

    def lists(self) -> Dict[str, object]:
        """Host copies of this step's lists and of the window state (synchronises)."""
        torch.cuda.synchronize(self.device)
        c = self.counts.cpu()
        na, ne, nm, nl, nh = (int(c[i]) for i in (B.CNT_N_ACTIVE, B.CNT_N_EVICT, B.CNT_N_MOVES,
                                                  B.CNT_N_LOAD, B.CNT_N_HITS))
        F, cap = self.d_ff, self.capacity
        out = {
            "active_idx": self._view("active_idx", F)[:na], "evict_ids": self._view("evict_ids", cap)[:ne],
            "move_src": self._view("move_src", cap)[:nm], "move_dst": self._view("move_dst", cap)[:nm],
            "load_ids": self._view("load_ids", cap)[:nl], "load_slots": self._view("load_slots", cap)[:nl],
            "active_slots": self._view("active_slots", F)[:na], "hit_slots": self._view("hit_slots", F)[:nh],
            "pointers": self._view("pointers", cap), "slot_of": self._view("slot_of", F),
            "last_active": self._view("last_active", F),
            "bias": self._view("bias", cap, torch.float16),
        }
        if self.spec_keep > 0:
            out["keep_token"] = self._view("keep_token", F, torch.int8)
        out = {k: v.cpu().numpy() for k, v in out.items()}
        out.update(num_used_before=int(c[B.CNT_NUM_USED_BEFORE]), num_kept=int(c[B.CNT_NUM_KEPT]),
                   num_used=int(c[B.CNT_NUM_USED]), step=int(c[B.CNT_STEP]), status=int(c[B.CNT_STATUS]),
                   k_eff=int(c[B.CNT_K_EFF]))
        return out

    def close(self) -> None:
        if getattr(self, "handle", None):
            intact = self.guards_intact()
            B.lif_destroy_layer(self.handle)
            self.handle = None
            if not intact:
                raise RuntimeError("a kernel wrote past the end of the cache or of the workspace")

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def pinned_store(d_ff: int, d_model: int, n_vec: int = 2) -> torch.Tensor:
    """Pinned (and, under unified addressing, device-mapped) host tensor for one layer's
    bundle store, fp16 [d_ff][n_vec*d_model] (n_vec = 3 when the gate row is bundled)."""
    return torch.empty(d_ff, n_vec * d_model, dtype=torch.float16, pin_memory=True)


def neuron_shard(d_ff: int, rank: int, world: int):
    """Ids [lo, hi) of the neurons that device ``rank`` of ``world`` owns when one layer's
    neurons are split over several devices: equal contiguous shares, each a multiple of 8
    (the layer description's rule for d_ff)."""
    if world < 1 or not 0 <= rank < world or d_ff % (8 * world):
        raise ValueError(f"d_ff={d_ff} does not split into {world} shares that are multiples of 8")
    per = d_ff // world
    return rank * per, (rank + 1) * per


def sum_partial_outputs(y: torch.Tensor, group=None) -> torch.Tensor:
    """The one exchange of a neuron-sharded layer-step: every device holds the FFN terms of its
    own neurons in ``y`` (fp32 ``[n_streams][d_model]``); afterwards every device holds their
    sum.  In place, on the current stream (NCCL) or on the host (gloo).  One device: no-op."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(y, op=dist.ReduceOp.SUM, group=group)
    return y


class PeerExchange:
    """The exchange of a neuron-sharded token over peer-mapped device memory instead of a
    library all-reduce.  Every rank writes its partial output of layer l into slot l of a
    buffer that all ranks of the group have mapped (torch symmetric memory: allocation and
    address exchange only); after a barrier across the ranks, ``lif_sum_peer_outputs`` reads
    all ranks' slots with plain loads and adds them in rank order, so every rank gets the same
    bits.  A slot is rewritten only in the next token, after ``end_token``'s barrier, so one
    barrier per layer is enough.  Call the methods with the compute stream current."""

    def __init__(self, n_layers: int, n_streams: int, d_model: int, device, group=None):
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm
        group = group if group is not None else dist.group.WORLD
        self.partials = symm.empty(n_layers, n_streams, d_model, dtype=torch.float32,
                                   device=torch.device(device))
        self.handle = symm.rendezvous(self.partials, group)
        self.slot_bytes = n_streams * d_model * 4
        self.peer_ptrs = [int(p) for p in self.handle.buffer_ptrs]     # rank order
        assert self.peer_ptrs[self.handle.rank] == self.partials.data_ptr()

    def sum_layer(self, l: int, y: torch.Tensor, stream=None) -> None:
        """y = sum over ranks of slot l, once every rank's slot l is complete."""
        self.handle.barrier(channel=0)
        B.lif_sum_peer_outputs([p + l * self.slot_bytes for p in self.peer_ptrs], y, stream)

    def end_token(self) -> None:
        """No rank starts the next token (and rewrites its slots) while a peer still reads."""
        self.handle.barrier(channel=1)


def build_stack(cfg, device="cuda:0", n_layers: Optional[int] = None, capacity_margin: float = 8.0,
                ffn_mode: int = 0, gen_device=None, gate_mode: int = 0, activation: int = 0,
                activation_threshold: float = 0.0, append_first: int = 0,
                shard=None, bias_down: Optional[List[torch.Tensor]] = None) -> List[Layer]:
    """Generate the weights of a named synthetic configuration and create its layers.

    ``shard = (rank, world)`` keeps only this device's share of every layer's neurons (its rows
    of the bundle store, its predictor columns, offsets and biases, a window cache sized for its
    share): the layer's output is then the sum over devices of the outputs computed here
    (``sum_partial_outputs``).  ``bias_down`` (one fp16 ``[d_model]`` tensor per layer) is given
    to the first device only, so that the sum holds it once."""
    from . import workloads as W
    layers = []
    gen_device = gen_device or device
    n_vec = 3 if gate_mode == B.GATE_BUNDLED else 2
    for l in range(n_layers or cfg.n_layers):
        if shard is None:
            lo, hi = 0, cfg.d_ff
            store = pinned_store(cfg.d_ff, cfg.d_model, n_vec)
            w = W.make_layer(cfg, l, device=gen_device, bundles_out=store, gate_mode=gate_mode,
                             act_threshold=activation_threshold)
        else:
            lo, hi = neuron_shard(cfg.d_ff, *shard)
            w = W.slice_layer(W.make_layer(cfg, l, device=gen_device, gate_mode=gate_mode,
                                           act_threshold=activation_threshold), lo, hi)
            store = pinned_store(hi - lo, cfg.d_model, n_vec)
            store.copy_(w["bundles"])
        cap = min(hi - lo, W.window_capacity(cfg, w["p"], capacity_margin))
        dev = lambda t: None if t is None else t.to(device).contiguous()
        b_down = bias_down[l] if bias_down is not None and (shard is None or shard[0] == 0) else None
        layers.append(Layer(d_model=cfg.d_model, d_ff=hi - lo, rank=cfg.rank, window_k=cfg.window_k,
                            capacity=cap, host_bundles=store, pred_A=dev(w["A"]), pred_B=dev(w["B"]),
                            pred_c=dev(w["c"]), bias_up=dev(w["bias_up"]), bias_down=dev(b_down),
                            n_streams=cfg.n_streams,
                            ffn_mode=ffn_mode, gate_mode=gate_mode, gate=dev(w.get("gate")),
                            activation=activation, activation_threshold=activation_threshold,
                            append_first=append_first, device=device))
    return layers
