"""Seeded synthetic workloads for the sparse-decode hot path.

This module only *generates inputs*: weights in row-column bundle layout, predictor
factors, per-neuron offsets, and auto-regressive decode inputs.  It contains none of the
method's arithmetic (no predictor, no window logic, no FFN) and is the one module that both
the CUDA path and the CPU checker are fed from.

The five named configurations stand in for trained ReLU models decoding a text corpus
(the paper's Section 4 setup); the recipe is:

* bundle ``i`` = up-projection row ``i`` followed by down-projection column ``i``
  (Section 3.2, "Bundling Columns and Rows"), entries ~ N(0, 0.02^2), stored fp16;
* neuron popularity ``p_i = min(0.95, s * exp(sigma * g_i))`` with ``g_i ~ N(0, 1)`` and ``s``
  found by bisection so that ``mean(p) = mean_fire``;
* up-projection bias ``b_i = ||w_i|| * Phi^-1(p_i)`` so a N(0, I) input fires neuron ``i`` with
  probability ``p_i``;
* low-rank predictor factors ``A[d][r]``, ``B[r][F]`` ~ N(0, 1) with unit-norm columns, so a
  N(0, I) input gives N(0, 1) scores; per-neuron offset ``c_i = Phi^-1(p_i)``, threshold 0;
* decode inputs ``x_t = rho * x_{t-1} + noise * eps_t``, ``x_0, eps_t ~ N(0, I)``, fp16;
* gated layers (Appendix C, Llama 2): a gate row per neuron drawn like the up row; the bias
  ``b_i = threshold + ||gate_i|| * Phi^-1(p_i)`` makes the gate value pass the activation's
  threshold with probability ``p_i``; bundle = gate | up | down, or up | down with the gate
  rows returned apart as the resident gate projection.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Dict, Optional

import torch


@dataclass(frozen=True)
class LifConfig:
    name: str
    n_layers: int
    d_model: int
    d_ff: int
    rank: int
    window_k: int
    n_streams: int
    steps: int
    mean_fire: float      # mean per-stream firing probability
    sigma_pop: float      # sigma of the lognormal popularity
    rho: float            # AR(1) coefficient of the decode inputs
    noise: float          # AR(1) innovation scale
    seed: int

    @property
    def bundle_bytes(self) -> int:
        return 2 * self.d_model * 2

    def scaled(self, **kw) -> "LifConfig":
        return replace(self, **kw)


def _ar_noise(rho: float) -> float:
    return math.sqrt(1.0 - rho * rho)


CONFIGS: Dict[str, LifConfig] = {
    "tiny": LifConfig("tiny", 2, 256, 1024, 16, 5, 1, 32, 0.05, 1.0, 0.8, 0.6, 0),
    "opt6p7b": LifConfig("opt6p7b", 32, 4096, 16384, 128, 5, 1, 128, 0.03, 1.0, 0.9,
                         _ar_noise(0.9), 1),
    "falcon7b": LifConfig("falcon7b", 32, 4544, 18176, 128, 5, 1, 256, 0.05, 1.5, 0.85,
                          _ar_noise(0.85), 2),
    "phi2": LifConfig("phi2", 32, 2560, 10240, 64, 4, 1, 256, 0.10, 1.0, 0.7,
                      _ar_noise(0.7), 3),
    "batched8": LifConfig("batched8", 48, 7168, 28672, 256, 5, 8, 64, 0.03, 1.0, 0.9,
                          _ar_noise(0.9), 4),
    # gated FFN of Appendix C (Llama 2 7B shapes: sparsity above 90 %, window of 2, rank 256)
    "llama2_7b": LifConfig("llama2_7b", 32, 4096, 11008, 256, 2, 1, 64, 0.08, 1.0, 0.9,
                           _ar_noise(0.9), 5),
}


def _generator(device: torch.device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def popularity(cfg: LifConfig, layer: int) -> torch.Tensor:
    """Per-neuron firing probability p_i (float64, CPU), clipped lognormal with the
    configured mean."""
    g = _generator(torch.device("cpu"), cfg.seed * 1000 + layer)
    gi = torch.randn(cfg.d_ff, generator=g, dtype=torch.float64)
    e = torch.exp(cfg.sigma_pop * gi)
    lo, hi = 0.0, 1.0
    for _ in range(80):
        mid = 0.5 * (lo + hi)
        if torch.clamp(mid * e, max=0.95).mean().item() < cfg.mean_fire:
            lo = mid
        else:
            hi = mid
    return torch.clamp(0.5 * (lo + hi) * e, max=0.95)


GATE_NONE, GATE_BUNDLED, GATE_RESIDENT = range(3)


def make_layer(cfg: LifConfig, layer: int, device: Optional[torch.device] = None,
               bundles_out: Optional[torch.Tensor] = None, gate_mode: int = GATE_NONE,
               act_threshold: float = 0.0) -> Dict[str, torch.Tensor]:
    """Generate one layer.  Random draws run on ``device`` (Philox on CUDA, MT on CPU; a run
    feeds the same tensors to every consumer, so the two never need to agree).  ``bundles_out``
    (fp16 ``[F][2d]``, typically a pinned host tensor) receives the bundle store; otherwise
    the bundles stay on ``device``.  ``gate_mode``: GATE_BUNDLED gives ``[F][3d]`` bundles
    (gate | up | down), GATE_RESIDENT ``[F][2d]`` bundles (up | down) plus ``gate`` ``[F][d]``;
    in both ``bias_up`` is the gate's bias, placed so that the gate value passes
    ``act_threshold`` with probability p_i."""
    device = torch.device(device or "cpu")
    d, F, r = cfg.d_model, cfg.d_ff, cfg.rank
    g = _generator(device, cfg.seed * 1000 + layer + 500)
    p = popularity(cfg, layer)
    q = torch.special.ndtri(p)                                        # Phi^-1(p_i), float64

    drawn = 2 if gate_mode == GATE_NONE else 3                        # vectors drawn per neuron
    stored = 2 if gate_mode != GATE_BUNDLED else 3                    # vectors per bundle
    bundles = torch.empty(F, stored * d, dtype=torch.float16, device=device)
    gate = torch.empty(F, d, dtype=torch.float16, device=device) if gate_mode == GATE_RESIDENT else None
    norms = torch.empty(F, dtype=torch.float64, device=device)
    rows = max(1, min(F, (64 << 20) // (drawn * d)))                  # ~256 MB fp32 scratch
    for i0 in range(0, F, rows):
        i1 = min(F, i0 + rows)
        blk = (torch.randn(i1 - i0, drawn * d, generator=g, device=device, dtype=torch.float32)
               * 0.02).to(torch.float16)
        if gate is None:
            bundles[i0:i1] = blk
        else:
            gate[i0:i1] = blk[:, :d]
            bundles[i0:i1] = blk[:, d:]
        norms[i0:i1] = blk[:, :d].double().square().sum(dim=1).sqrt()
    bias_up = (norms * q.to(device) + act_threshold).to(torch.float16)

    A = torch.randn(d, r, generator=g, device=device, dtype=torch.float32)
    A = (A / A.norm(dim=0, keepdim=True)).to(torch.float16)
    B = torch.randn(r, F, generator=g, device=device, dtype=torch.float32)
    B = (B / B.norm(dim=0, keepdim=True)).to(torch.float16)
    c = q.to(torch.float32).to(device)

    out = {"bias_up": bias_up, "A": A.contiguous(), "B": B.contiguous(), "c": c, "p": p}
    if gate is not None:
        out["gate"] = gate
    if bundles_out is not None:
        bundles_out.copy_(bundles)
        out["bundles"] = bundles_out
    else:
        out["bundles"] = bundles
    return out


def slice_layer(w: Dict[str, torch.Tensor], lo: int, hi: int) -> Dict[str, torch.Tensor]:
    """The tensors of neurons ``lo`` .. ``hi - 1`` of a generated layer, as contiguous copies:
    rows of the bundle store (and of the gate projection), columns of the predictor's second
    factor, the per-neuron offsets, biases and popularities.  The first factor ``A`` is shared
    by every neuron and returned as it is.  Slicing only: no arithmetic."""
    per_neuron_rows = ("bundles", "gate", "bias_up", "c", "p")
    out = {}
    for name, t in w.items():
        if name in per_neuron_rows:
            out[name] = t[lo:hi].contiguous()
        elif name == "B":
            out[name] = t[:, lo:hi].contiguous()
        else:
            out[name] = t
    return out


def make_inputs(cfg: LifConfig, device: Optional[torch.device] = None) -> torch.Tensor:
    """Decode inputs ``X[steps][n_streams][d_model]`` fp16: independent AR(1) sequences."""
    device = torch.device(device or "cpu")
    g = _generator(device, cfg.seed * 1000 + 999)
    S, d = cfg.n_streams, cfg.d_model
    x = torch.randn(S, d, generator=g, device=device, dtype=torch.float32)
    out = torch.empty(cfg.steps, S, d, dtype=torch.float16, device=device)
    for t in range(cfg.steps):
        if t > 0:
            x = cfg.rho * x + cfg.noise * torch.randn(S, d, generator=g, device=device,
                                                      dtype=torch.float32)
        out[t] = x.to(torch.float16)
    return out


def window_capacity(cfg: LifConfig, p: torch.Tensor, margin_sigmas: float = 8.0) -> int:
    """Rows to pre-allocate for one layer's window cache (the paper's Req_i, Section 3.3):
    the expected union of ``window_k * n_streams`` independent draws of the active set plus a
    ``margin_sigmas`` binomial margin, rounded up to a multiple of 64.  Temporal correlation of
    the inputs only makes the true union smaller."""
    n_draws = cfg.window_k * cfg.n_streams
    hit = 1.0 - (1.0 - p.double()) ** n_draws
    mean = hit.sum().item()
    var = (hit * (1.0 - hit)).sum().item()
    cap = int(math.ceil(mean + margin_sigmas * math.sqrt(var))) + 64
    return min(cfg.d_ff, (cap + 63) // 64 * 64)
