"""Seeded synthetic model-shaped tensors for the sensitivity sweep.

The paper measures on ImageNet-trained networks with 100 calibration images; neither the
data nor the weights are available, so tensors with the same shapes and with plausible value
distributions stand in for them.  This module draws values only -- it contains none of the
method's arithmetic (no ranges, scales, codes or metrics) and is the one module that both the
CPU oracle's tests and the CUDA path's tests/bench import.  Both sides always consume the
*same bytes*: tensors are drawn once, on one device, and copied to wherever the other side
needs them.

Recipe (per config, see ``CONFIGS``):
  weights      Kaiming-normal N(0, 2/fan_in) times a per-output-channel multiplier
               lognormal(0, ch_sigma); optionally a fraction ``outlier_frac`` of the weights is
               replaced by +-outlier_k standard deviations.
  reference    per channel s_c ~ lognormal(0, 0.5); x drawn from the layer's ``act``
  activations  distribution ("relu", "relu6", "half", "gauss", see gen.models).
  quantized-   y = x + N(0, 0.01 * (1 + layer_idx/8) * s_c): noise that grows with depth, a
  pass acts    stand-in for the accumulated quantization noise of a real int8 pass.
Sub-seeds: every tensor gets its own torch.Generator seeded with mix(seed, layer, kind), so
a layer's tensors do not depend on which other layers were generated.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import torch

from .models import SHAPES, LayerShape


@dataclass(frozen=True)
class SynthConfig:
    name: str
    shapes: str
    batch: int
    w_granularity: Sequence[str]      # each of "tensor" | "channel"; all are scored, first is ranked
    a_range: str                      # "minmax" | "percentile"
    a_percentile: float = 0.9999
    ch_sigma: float = 0.3
    outlier_frac: float = 0.0
    outlier_k: float = 0.0
    bops_rate_permyriad: int = 4000   # requested BOPs-reduction rate for the layer-set selection


# The five workloads, in the order the benchmark description lists them.
CONFIGS: Dict[str, SynthConfig] = {
    "squeezenet": SynthConfig("squeezenet", "squeezenet", 1, ("tensor",), "minmax"),
    "resnet18": SynthConfig("resnet18", "resnet18", 32, ("channel",), "percentile",
                            outlier_frac=1e-3, outlier_k=8.0),
    "resnet50": SynthConfig("resnet50", "resnet50", 64, ("channel",), "minmax"),
    "mobilenetv2": SynthConfig("mobilenetv2", "mobilenetv2", 128, ("channel", "tensor"),
                               "percentile", ch_sigma=1.5),
    "vgg16": SynthConfig("vgg16", "vgg16", 64, ("channel",), "percentile",
                         outlier_frac=1e-3, outlier_k=10.0),
}
CONFIG_ORDER = ["squeezenet", "resnet18", "resnet50", "mobilenetv2", "vgg16"]


@dataclass
class SynthLayer:
    shape: LayerShape
    index: int
    w: torch.Tensor                   # [cout, K] fp32
    x: torch.Tensor                   # [B, cout, hw*hw] fp32, reference-pass output
    y: torch.Tensor                   # same shape, quantized-pass output
    macs: int


@dataclass
class SynthModel:
    config: SynthConfig
    batch: int
    seed: int
    layers: List[SynthLayer] = field(default_factory=list)

    @property
    def weight_elems(self) -> int:
        return sum(l.w.numel() for l in self.layers)

    @property
    def act_elems(self) -> int:
        return sum(l.x.numel() for l in self.layers)


_M64 = (1 << 64) - 1


def _mix(*vals: int) -> int:
    """splitmix64-style integer mixing of a tuple into one 63-bit seed."""
    h = 0x9E3779B97F4A7C15
    for v in vals:
        h = (h + (v & _M64) + 0x9E3779B97F4A7C15) & _M64
        h = ((h ^ (h >> 30)) * 0xBF58476D1CE4E5B9) & _M64
        h = ((h ^ (h >> 27)) * 0x94D049BB133111EB) & _M64
        h ^= h >> 31
    return h & ((1 << 63) - 1)


def _gen(device, *key: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_mix(*key))
    return g


def draw_weights(shape: LayerShape, cfg: SynthConfig, seed: int, layer_idx: int, device) -> torch.Tensor:
    g = _gen(device, seed, layer_idx, 1)
    std = math.sqrt(2.0 / shape.k_elems)
    w = torch.randn(shape.cout, shape.k_elems, generator=g, device=device, dtype=torch.float32)
    mult = torch.exp(cfg.ch_sigma * torch.randn(shape.cout, 1, generator=g, device=device,
                                                dtype=torch.float32))
    w.mul_(std).mul_(mult)
    if cfg.outlier_frac > 0.0:
        pick = torch.rand(w.shape, generator=g, device=device) < cfg.outlier_frac
        sign = torch.where(torch.rand(w.shape, generator=g, device=device) < 0.5, -1.0, 1.0)
        w = torch.where(pick, sign * (cfg.outlier_k * std), w)
    return w.contiguous()


def draw_activations(shape: LayerShape, batch: int, seed: int, layer_idx: int, device):
    """Returns (x, y): reference-pass and quantized-pass outputs, [batch, cout, hw*hw]."""
    g = _gen(device, seed, layer_idx, 2)
    hw2 = shape.out_hw * shape.out_hw
    s_c = torch.exp(0.5 * torch.randn(1, shape.cout, 1, generator=g, device=device,
                                      dtype=torch.float32))
    x = torch.randn(batch, shape.cout, hw2, generator=g, device=device, dtype=torch.float32)
    x.mul_(s_c)
    if shape.act == "relu":
        x.clamp_(min=0.0)
    elif shape.act == "relu6":
        x.clamp_(min=0.0, max=6.0)
    elif shape.act == "half":
        x.abs_()
    elif shape.act != "gauss":
        raise ValueError(f"unknown activation distribution {shape.act!r}")
    g2 = _gen(device, seed, layer_idx, 3)
    y = torch.randn(batch, shape.cout, hw2, generator=g2, device=device, dtype=torch.float32)
    y.mul_(s_c * (0.01 * (1.0 + layer_idx / 8.0))).add_(x)
    return x.contiguous(), y.contiguous()


def make_model(name: str, seed: int = 0, device="cpu", batch: Optional[int] = None,
               layer_indices: Optional[Sequence[int]] = None) -> SynthModel:
    """Draw every tensor of one workload.  ``batch`` overrides the config's batch size (the
    tests shrink it so the CPU oracle finishes in seconds); ``layer_indices`` keeps a subset of
    layers, each still seeded by its index in the full model."""
    cfg = CONFIGS[name]
    shapes = SHAPES[cfg.shapes]()
    b = cfg.batch if batch is None else int(batch)
    model = SynthModel(cfg, b, seed)
    idxs = range(len(shapes)) if layer_indices is None else layer_indices
    for i in idxs:
        sh = shapes[i]
        w = draw_weights(sh, cfg, seed, i, device)
        x, y = draw_activations(sh, b, seed, i, device)
        model.layers.append(SynthLayer(sh, i, w, x, y, sh.macs))
    return model


def model_sizes(name: str, batch: Optional[int] = None):
    """(weight elements, activation elements per pass, number of layers) without drawing anything."""
    cfg = CONFIGS[name]
    shapes = SHAPES[cfg.shapes]()
    b = cfg.batch if batch is None else int(batch)
    w = sum(s.weight_elems for s in shapes)
    a = sum(s.act_elems_per_image for s in shapes) * b
    return w, a, len(shapes)


def swept_bytes(name: str, batch: Optional[int] = None) -> int:
    """Algorithmic bytes one full sensitivity pass must read: every weight element twice
    (range pass, metric pass) per scored granularity, every activation element in the range
    pass (4 B), the histogram pass when percentile clipping is on (4 B) and the paired metric
    pass over x and y (8 B)."""
    cfg = CONFIGS[name]
    w, a, _ = model_sizes(name, batch)
    a_bytes = 16 if cfg.a_range == "percentile" else 12
    return 8 * w * len(cfg.w_granularity) + a_bytes * a
