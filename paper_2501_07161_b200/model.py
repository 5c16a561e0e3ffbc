"""Descriptor marshalling for a whole model: weights first, then activations, then any extra
weight scorings -- the layout qv2_sweep_model expects."""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import torch

from . import binding as B


@dataclass
class ModelDescs:
    descs: object                 # ctypes array of TensorDesc
    n_layers: int
    n_tensors: int
    macs: torch.Tensor            # int64 [n_layers] on the tensors' device
    keepalive: List[torch.Tensor]
    rate_permyriad: int


def model_descs(model, host: bool = False, act_granularity: str = "tensor") -> ModelDescs:
    """`model` is any object with `.layers` (each with w [cout,K], x and y [B,C,HW], macs) and
    `.config` (w_granularity, a_range, a_percentile, bops_rate_permyriad).  The paper's set-ups
    quantize activations per tensor; act_granularity="channel" is the per-channel variant, with
    one percentile clip per channel where the configuration clips at all."""
    cfg = model.config
    gran = {"tensor": B.PER_TENSOR, "channel": B.PER_CHANNEL}
    a_range = B.PERCENTILE if cfg.a_range == "percentile" else B.MINMAX
    if a_range == B.PERCENTILE and act_granularity == "channel":
        a_range = B.PERCENTILE_GROUP
    descs, keep = [], []
    L = model.layers
    for l in L:
        descs.append(B.make_desc(l.w, None, 1, l.w.shape[0], l.w.shape[1], gran[cfg.w_granularity[0]],
                                 B.SYM_I8, B.ABSMAX))
        keep.append(l.w)
    for l in L:
        b, c, hw = l.x.shape
        descs.append(B.make_desc(l.x, l.y, b, c, hw, gran[act_granularity], B.ASYM_U8, a_range,
                                 cfg.a_percentile if a_range != B.MINMAX else 0.0))
        keep += [l.x, l.y]
    for g in cfg.w_granularity[1:]:
        for l in L:
            descs.append(B.make_desc(l.w, None, 1, l.w.shape[0], l.w.shape[1], gran[g], B.SYM_I8, B.ABSMAX))
    dev = L[0].w.device if not host else torch.device("cpu")
    macs = torch.tensor([l.macs for l in L], dtype=torch.int64, device=dev)
    return ModelDescs(B.desc_array(descs), len(L), len(descs), macs, keep, cfg.bops_rate_permyriad)
