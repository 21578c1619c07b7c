"""Seeded synthetic inputs shaped like the paper's Infinity workloads.

This module only draws random tensors and names workload shapes; it holds none of the
method's arithmetic, so both the CUDA path and the CPU oracle may be fed from it.  The
real activations need model weights and captions that are not available here; the recipe
below stands in for them:

* Q, V ~ N(0, I).
* K[pos] = mu_{scale(pos)} + N(0, I) with a per-slice, per-scale offset mu_k ~ N(0, 0.5^2 I),
  so that attention is peaked within scales.
* 4 "sink" keys per slice (position 0 plus 3 seeded positions below T_c) have their rows
  multiplied by 4.
* planted layer roles (workloads with n_drafters > 0): refiner layers get Q_k += mu_k, which
  lifts the logits of their own scale (concentrated, local attention); drafter layers get
  Q_k *= 0.25, a high softmax temperature that disperses attention over the whole history.
  This gives the offline layer statistics a known answer.

Everything is a pure function of (seed, layer, scale): tensors for one (layer, scale) can be
regenerated at any time, in any order, on the same device type.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

SIDES_4 = (1, 2, 4, 8)
SIDES_13 = (1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64)
SIDES_16 = SIDES_13 + (80, 96, 128)
SIDES_19 = SIDES_16 + (160, 192, 256)      # a 4K-class image at the same 16 x downsampling: 170 521 tokens


@dataclass
class Workload:
    name: str
    n_layers: int
    batch: int
    n_heads: int
    head_dim: int
    dtype: str  # "bf16" | "f32"
    sides: tuple
    seed: int
    planted: bool = True
    n_drafters: int = 0          # layers planted as drafters
    drafter_pct: float = 0.30
    refiner_pct: float = 0.03
    window: int = 16
    extra: dict = field(default_factory=dict)

    @property
    def n_scales(self):
        return len(self.sides)

    @property
    def n_tokens(self):
        return [s * s for s in self.sides]

    @property
    def n_slices(self):
        return self.n_layers * self.batch * self.n_heads


WORKLOADS = {
    # configs[0]: tiny fp32 case, window = whole current map, budget 16
    "tiny": Workload("tiny", 1, 1, 4, 64, "f32", SIDES_4, seed=1, planted=False, window=64),
    # configs[1]: one 2B-class layer
    "layer2b": Workload("layer2b", 1, 8, 16, 128, "bf16", SIDES_13, seed=2),
    # configs[2]: the 32-layer 2B-class pass, 8 drafters / 24 refiners (headline)
    "pass2b": Workload("pass2b", 32, 8, 16, 128, "bf16", SIDES_13, seed=3, n_drafters=8),
    # configs[3]: the 40-layer 8B-class pass, 10 / 30
    "pass8b": Workload("pass8b", 40, 8, 32, 128, "bf16", SIDES_13, seed=4, n_drafters=10),
    # configs[4]: 16-scale stress
    "hires": Workload("hires", 32, 4, 16, 128, "bf16", SIDES_16, seed=5, n_drafters=8),
    # the headline pass with the batch doubled, as under classifier-free guidance (a conditional and an
    # unconditional branch per image run through the same layers)
    # beyond configs[4]: the "ultra-high resolutions such as 4K" the paper names as the method's target (Sec. 4.3):
    # 19 scales up to 256 x 256; a slice outgrows one CTA's shared memory, so select and compact work from global memory
    "uhd4k": Workload("uhd4k", 32, 1, 16, 128, "bf16", SIDES_19, seed=7, n_drafters=8),
    "pass2b_cfg": Workload("pass2b_cfg", 32, 16, 16, 128, "bf16", SIDES_13, seed=6, n_drafters=8),
}


def torch_dtype(name):
    return {"bf16": torch.bfloat16, "f32": torch.float32}[name]


def _mix(*xs):
    """Small integer mixer for seeds (not part of the method)."""
    h = 0x9E3779B97F4A7C15
    for x in xs:
        h ^= (int(x) + 0x9E3779B97F4A7C15 + ((h << 6) & 0xFFFFFFFFFFFFFFFF) + (h >> 2)) & 0xFFFFFFFFFFFFFFFF
        h = (h * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
    return h & 0x7FFFFFFFFFFFFFFF


def drafter_layers(wl: Workload):
    """The seeded subset of layers planted as drafters (gamma = 0)."""
    if wl.n_drafters <= 0:
        return []
    g = torch.Generator(device="cpu")
    g.manual_seed(_mix(wl.seed, 0xD7A))
    return sorted(torch.randperm(wl.n_layers, generator=g)[: wl.n_drafters].tolist())


def sink_positions(wl: Workload, layer: int):
    """[B, H, 4] int64 (CPU): position 0 plus 3 distinct seeded positions in [1, T_c)."""
    n = wl.n_tokens
    t_c = sum(n[:-1])
    g = torch.Generator(device="cpu")
    g.manual_seed(_mix(wl.seed, layer, 0x51))
    out = torch.zeros(wl.batch, wl.n_heads, 4, dtype=torch.int64)
    if t_c > 4:
        r = torch.rand(wl.batch, wl.n_heads, t_c - 1, generator=g)
        out[..., 1:] = r.topk(3, dim=-1).indices + 1
    return out


def scale_inputs(wl: Workload, layer: int, scale: int, device="cpu"):
    """Q, K, V of scale `scale` (0-based) for one layer: each [B, H, n_k, d] in wl.dtype."""
    n = wl.n_tokens
    nk, d = n[scale], wl.head_dim
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(_mix(wl.seed, layer, scale, 0xA11))
    shape = (wl.batch, wl.n_heads, nk, d)
    Q = torch.randn(shape, generator=g, device=dev, dtype=torch.float32)
    K = torch.randn(shape, generator=g, device=dev, dtype=torch.float32)
    V = torch.randn(shape, generator=g, device=dev, dtype=torch.float32)
    if wl.planted:
        mu = 0.5 * torch.randn((wl.batch, wl.n_heads, 1, d), generator=g, device=dev, dtype=torch.float32)
        K += mu
        if wl.n_drafters > 0:
            if layer in drafter_layers(wl):
                Q *= 0.25
            else:
                Q += mu
        base = sum(n[:scale])
        sinks = sink_positions(wl, layer).to(dev) - base          # [B, H, 4] relative to this map
        inside = (sinks >= 0) & (sinks < nk)
        if bool(inside.any()):
            gain = torch.ones((wl.batch, wl.n_heads, nk), device=dev, dtype=torch.float32)
            bi, hi, si = torch.nonzero(inside, as_tuple=True)
            gain[bi, hi, sinks[bi, hi, si]] = 4.0
            K *= gain.unsqueeze(-1)
    dt = torch_dtype(wl.dtype)
    return Q.to(dt), K.to(dt), V.to(dt)
