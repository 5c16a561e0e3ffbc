"""Shared machinery of the GPU parity tests: run the same tensors through the CUDA library (via
its C ABI) and through the CPU oracle, and compare element by element.

Bars: ranges, parameters, histograms, clips, non-finite counts, codes and rank outputs are
bit-exact; MSE agrees within 1e-5 relative and SQNR within 1e-3 dB."""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

import oracle
import paper_2501_07161_b200 as q

MSE_RTOL = 1e-5
SQNR_ATOL_DB = 1e-3


@dataclass
class Spec:
    x: torch.Tensor                    # CPU or CUDA, fp32, flat or shaped; viewed [outer][channels][inner]
    outer: int
    channels: int
    inner: int
    per_channel: bool = False
    asym: bool = False
    percentile: Optional[float] = None
    y: Optional[torch.Tensor] = None
    raw: bool = False
    name: str = ""
    bits: int = 8
    dtype: torch.dtype = torch.float32  # element type the GPU side stores x and y in
    zp: bool = False                   # affine scheme with an integer zero point (implies asym)
    group_pct: bool = False            # percentile clip per channel (own histogram per group)


def bits(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def to_dev(t: Optional[torch.Tensor], misalign: int = 0, dtype: torch.dtype = torch.float32):
    """Copy to the GPU; `misalign` (0..3) shifts the start by that many elements past a
    256-byte boundary so that vector loads need a scalar head."""
    if t is None:
        return None
    flat = t.reshape(-1).to(dtype)
    if misalign == 0:
        return flat.cuda().contiguous()
    buf = torch.empty(flat.numel() + misalign, dtype=dtype, device="cuda")
    buf[misalign:].copy_(flat)
    return buf[misalign:]


def make_descs(specs: List[Spec], dev_x, dev_y, store_codes=True):
    descs = []
    for s, dx, dy in zip(specs, dev_x, dev_y):
        flags = (q.PAIR_RAW if s.raw else 0) | (q.STORE_CODES if store_codes and not s.raw and s.bits <= 8 else 0)
        descs.append(q.make_desc(dx, dy, s.outer, s.channels, s.inner,
                                 q.PER_CHANNEL if s.per_channel else q.PER_TENSOR,
                                 q.ASYM_U8_ZP if s.zp else (q.ASYM_U8 if s.asym else q.SYM_I8),
                                 (q.PERCENTILE_GROUP if s.group_pct else q.PERCENTILE) if s.percentile is not None else (q.MINMAX if (s.asym or s.zp) else q.ABSMAX),
                                 s.percentile or 0.0, flags, s.bits))
    return q.desc_array(descs)


def oracle_tensor(s: Spec, want_codes=True):
    # the oracle sees exactly the values the GPU side stores: rounded to the storage type, widened back
    x = s.x.detach().cpu().to(s.dtype).to(torch.float32).numpy().reshape(-1)
    y = None if s.y is None else s.y.detach().cpu().to(s.dtype).to(torch.float32).numpy().reshape(-1)
    mode = None
    if y is not None:
        mode = oracle.PAIR_RAW if s.raw else oracle.PAIR_REQUANT
    return oracle.sweep_tensor(x, y, s.outer, s.channels, s.inner, s.per_channel, 2 if s.zp else s.asym,
                               s.percentile, pair_mode=mode, want_codes=want_codes and not s.raw, bits=s.bits,
                               group_percentile=s.group_pct)


def assert_metric_close(got_mse, got_sqnr, ref_mse, ref_sqnr, what=""):
    if ref_mse == 0.0:
        assert got_mse == 0.0, f"{what}: mse {got_mse} != 0"
    else:
        assert abs(got_mse - ref_mse) <= MSE_RTOL * abs(ref_mse), \
            f"{what}: mse {got_mse} vs {ref_mse} rel {abs(got_mse - ref_mse) / abs(ref_mse):.3e}"
    if math.isinf(ref_sqnr):
        assert got_sqnr == ref_sqnr, f"{what}: sqnr {got_sqnr} vs {ref_sqnr}"
    else:
        assert abs(got_sqnr - ref_sqnr) <= SQNR_ATOL_DB, f"{what}: sqnr {got_sqnr} vs {ref_sqnr}"


def check_specs(ctx, specs: List[Spec], misalign_x=0, misalign_y=0, check_codes=True,
                twice=True):
    """Calibrate + measure every spec in ONE batched call each, compare with the oracle."""
    dev_x = [to_dev(s.x, misalign_x, s.dtype) for s in specs]
    dev_y = [to_dev(s.y, misalign_y, s.dtype) for s in specs]
    descs = make_descs(specs, dev_x, dev_y, store_codes=check_codes)
    want_group = any(s.group_pct for s in specs)
    cal = ctx.calibrate(descs, want_group=want_group)
    codes = None
    if check_codes:
        codes = [None if s.raw else torch.full((max(s.x.numel(), 1),), 0x55, dtype=torch.uint8, device="cuda")
                 for s in specs]
    met = ctx.quant_metrics(descs, cal.step, cal.inv, cal.offset, codes)
    torch.cuda.synchronize()
    if twice:
        cal2 = ctx.calibrate(descs)
        met2 = ctx.quant_metrics(descs, cal2.step, cal2.inv, cal2.offset, codes)
        torch.cuda.synchronize()
        for a, b in ((met.sse, met2.sse), (met.sig, met2.sig), (met.sqnr_db, met2.sqnr_db)):
            assert np.array_equal(a.cpu().numpy().view(np.uint64), b.cpu().numpy().view(np.uint64)), \
                "two runs differ"
    g = 0
    gh = 0                     # running index into the per-group histograms
    hist = cal.hist.cpu().numpy().view(np.uint64).reshape(-1, q.HIST_BINS)
    if want_group:
        ghist = cal.group_hist.cpu().numpy().view(np.uint64).reshape(-1, q.HIST_BINS)
        gclip = cal.group_clip.cpu().numpy()
    for t, s in enumerate(specs):
        ref = oracle_tensor(s, want_codes=check_codes)
        ng = s.channels if s.per_channel else 1
        sl = slice(g, g + ng)
        name = s.name or f"tensor{t}"
        for field in ("gmin", "gmax", "gabsmax", "step", "inv", "offset"):
            got = getattr(cal, field)[sl].cpu().numpy()
            exp = getattr(ref, field)
            assert np.array_equal(bits(got), bits(exp)), f"{name}: {field} differs: {got[:4]} vs {exp[:4]}"
        assert int(cal.nonfinite[t]) == ref.nonfinite, f"{name}: nonfinite"
        assert bits(cal.clip[t:t + 1].cpu().numpy())[0] == bits([ref.clip])[0], \
            f"{name}: clip {float(cal.clip[t])} vs {ref.clip}"
        if want_group:
            assert np.array_equal(bits(gclip[sl]), bits(ref.gclip)), f"{name}: group clips differ"
        if ref.ghist is not None:
            got = ghist[gh:gh + ng]
            assert np.array_equal(got, ref.ghist), \
                f"{name}: per-group histograms differ in groups {np.nonzero((got != ref.ghist).any(axis=1))[0][:8]}"
            assert not hist[t].any()
            gh += ng
        elif s.percentile is not None:
            assert np.array_equal(hist[t], ref.hist), f"{name}: histogram differs"
            assert int(hist[t].sum()) == s.x.numel() - ref.nonfinite
        else:
            assert not hist[t].any(), f"{name}: histogram of a non-percentile tensor must be zero"
        if ref.nonfinite == 0:
            assert_metric_close(float(met.mse[t]), float(met.sqnr_db[t]), ref.mse, ref.sqnr_db, name)
            if ref.sig > 0:
                assert abs(float(met.sig[t]) - ref.sig) <= MSE_RTOL * ref.sig, f"{name}: sig"
            if check_codes and not s.raw and s.x.numel() and s.bits <= 8:
                got = codes[t][: s.x.numel()].cpu().numpy()
                exp = ref.codes.view(np.uint8)
                nbad = int((got != exp).sum())
                assert nbad == 0, f"{name}: {nbad} codes differ"
        g += ng
    return cal, met
