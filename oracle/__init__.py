"""ctypes front end of the CPU oracle (``qv2_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke()`` and by the
``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``.  The CUDA package never imports it
and it never imports the CUDA package.  The arithmetic lives in the C file; this module only
marshals numpy arrays and strings the per-tensor steps together in the paper's order
(calibrate -> parameters -> fake-quantize and measure -> rank).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qv2_oracle.c")
_LIB = os.path.join(_HERE, "libqv2_oracle.so")
BINS = 2048

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc.  -ffp-contract=off keeps every multiply and add a separate,
    individually rounded operation."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = C.CDLL(build())
    f32p, u64p, f64p, u8p, u32p = (C.POINTER(C.c_float), C.POINTER(C.c_uint64),
                                   C.POINTER(C.c_double), C.POINTER(C.c_uint8),
                                   C.POINTER(C.c_uint32))
    lib.qv2o_ranges.argtypes = [f32p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_int,
                                f32p, f32p, f32p, u64p]
    lib.qv2o_ranges.restype = None
    lib.qv2o_histogram.argtypes = [f32p, C.c_uint64, C.c_float, u64p]
    lib.qv2o_histogram.restype = None
    lib.qv2o_percentile_clip.argtypes = [u64p, C.c_double, C.c_float]
    lib.qv2o_percentile_clip.restype = C.c_float
    lib.qv2o_qparams.argtypes = [C.c_int, C.c_int, C.c_float, C.c_uint64, f32p, f32p, f32p,
                                 f32p, f32p, f32p]
    lib.qv2o_qparams.restype = None
    lib.qv2o_quant_metrics.argtypes = [f32p, f32p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_int,
                                       C.c_int, C.c_int, f32p, f32p, f32p, u8p,
                                       f64p, f64p, f64p, f64p]
    lib.qv2o_quant_metrics.restype = None
    lib.qv2o_cosine.argtypes = [f32p, f32p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_int, C.c_int,
                                C.c_int, f32p, f32p, f32p]
    lib.qv2o_cosine.restype = C.c_double
    lib.qv2o_rank.argtypes = [C.c_uint32, f64p, f64p, f64p, f64p, u64p, f64p,
                              C.c_double, C.c_double, C.c_double, C.c_double,
                              C.c_int, C.c_uint32, C.c_uint32, u32p, u8p, u32p]
    lib.qv2o_rank.restype = None
    lib.qv2o_rank_ex.argtypes = [C.c_uint32, f64p, f64p, f64p, f64p, u64p, f64p,
                                 C.c_double, C.c_double, C.c_double, C.c_double,
                                 C.c_int, C.c_uint32, C.c_uint32, C.c_int, u32p, u8p, u32p]
    lib.qv2o_rank_ex.restype = None
    lib.qv2o_qparams_bits.argtypes = [C.c_int] + list(lib.qv2o_qparams.argtypes)
    lib.qv2o_qparams_bits.restype = None
    lib.qv2o_quant_metrics_bits.argtypes = [C.c_int] + list(lib.qv2o_quant_metrics.argtypes)
    lib.qv2o_quant_metrics_bits.restype = None
    lib.qv2o_cosine_bits.argtypes = [C.c_int] + list(lib.qv2o_cosine.argtypes)
    lib.qv2o_cosine_bits.restype = C.c_double
    lib.qv2o_kl_bits.argtypes = [C.c_int, f32p, f32p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_int, C.c_int,
                                 C.c_int, f32p, f32p, f32p, C.c_float, u64p, u64p]
    lib.qv2o_kl_bits.restype = C.c_double
    lib.qv2o_fold_batchnorm.argtypes = [f32p] * 6 + [C.c_uint64, C.c_uint64, f32p, f32p]
    lib.qv2o_fold_batchnorm.restype = None
    lib.qv2o_group_histograms.argtypes = [f32p, C.c_uint64, C.c_uint64, C.c_uint64, f32p, C.c_double, u64p, f32p]
    lib.qv2o_group_histograms.restype = None
    lib.qv2o_qparams_gclip.argtypes = [C.c_int, C.c_int, C.c_uint64, f32p, f32p, f32p, f32p, f32p, f32p, f32p]
    lib.qv2o_qparams_gclip.restype = None
    lib.qv2o_rank_fused.argtypes = [C.c_uint32, f64p, f64p, f64p, f64p, u64p, f64p, u32p,
                                    C.c_double, C.c_double, C.c_double, C.c_double,
                                    C.c_int, C.c_uint32, C.c_uint32, u32p, u8p, u32p]
    lib.qv2o_rank_fused.restype = None
    lib.qv2o_rank_fused_ex.argtypes = [C.c_uint32, f64p, f64p, f64p, f64p, u64p, f64p, u32p,
                                       C.c_double, C.c_double, C.c_double, C.c_double,
                                       C.c_int, C.c_uint32, C.c_uint32, C.c_int, u32p, u8p, u32p]
    lib.qv2o_rank_fused_ex.restype = None
    _lib = lib
    return lib


def _p(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


# ------------------------------------------------------------------------------ per-step calls
def ranges(x, outer: int, channels: int, inner: int, per_channel: bool):
    """-> (gmin, gmax, gabsmax, nonfinite) over the groups of x viewed [outer][channels][inner]."""
    lib = _load()
    x = _f32(x).reshape(-1)
    assert x.size == outer * channels * inner
    g = channels if per_channel else 1
    gmin = np.zeros(g, np.float32); gmax = np.zeros(g, np.float32); gabs = np.zeros(g, np.float32)
    bad = C.c_uint64(0)
    lib.qv2o_ranges(_p(x, C.c_float), outer, channels, inner, int(per_channel),
                    _p(gmin, C.c_float), _p(gmax, C.c_float), _p(gabs, C.c_float), C.byref(bad))
    return gmin, gmax, gabs, int(bad.value)


def histogram(x, absmax: float) -> np.ndarray:
    lib = _load()
    x = _f32(x).reshape(-1)
    hist = np.zeros(BINS, np.uint64)
    lib.qv2o_histogram(_p(x, C.c_float), x.size, C.c_float(absmax), _p(hist, C.c_uint64))
    return hist


def percentile_clip(hist: np.ndarray, p: float, absmax: float) -> np.float32:
    lib = _load()
    hist = np.ascontiguousarray(hist, dtype=np.uint64)
    return np.float32(lib.qv2o_percentile_clip(_p(hist, C.c_uint64), float(p), C.c_float(absmax)))


def qparams(asym_u8: bool, gmin, gmax, gabsmax, clip: Optional[float] = None, bits: int = 8):
    lib = _load()
    gmin, gmax, gabsmax = _f32(gmin), _f32(gmax), _f32(gabsmax)
    g = gmin.size
    step = np.zeros(g, np.float32); inv = np.zeros(g, np.float32); off = np.zeros(g, np.float32)
    lib.qv2o_qparams_bits(int(bits), int(asym_u8), int(clip is not None), C.c_float(0.0 if clip is None else clip),
                     g, _p(gmin, C.c_float), _p(gmax, C.c_float), _p(gabsmax, C.c_float),
                     _p(step, C.c_float), _p(inv, C.c_float), _p(off, C.c_float))
    return step, inv, off


def group_histograms(x, outer: int, channels: int, inner: int, gabsmax, p: float):
    """One |x| histogram and one percentile clip per channel of a [outer][channels][inner] tensor."""
    lib = _load()
    x = _f32(x).reshape(-1)
    assert x.size == outer * channels * inner
    gabsmax = _f32(gabsmax)
    assert gabsmax.size == channels
    hist = np.zeros((channels, BINS), np.uint64)
    clip = np.zeros(channels, np.float32)
    lib.qv2o_group_histograms(_p(x, C.c_float), outer, channels, inner, _p(gabsmax, C.c_float), float(p),
                              _p(hist, C.c_uint64), _p(clip, C.c_float))
    return hist, clip


def qparams_gclip(scheme, gmin, gmax, gabsmax, gclip, bits: int = 8):
    """qparams with one clip value per group."""
    lib = _load()
    gmin, gmax, gabsmax, gclip = _f32(gmin), _f32(gmax), _f32(gabsmax), _f32(gclip)
    g = gmin.size
    assert gclip.size == g
    step = np.zeros(g, np.float32); inv = np.zeros(g, np.float32); off = np.zeros(g, np.float32)
    lib.qv2o_qparams_gclip(int(bits), int(scheme), g, _p(gclip, C.c_float), _p(gmin, C.c_float),
                           _p(gmax, C.c_float), _p(gabsmax, C.c_float),
                           _p(step, C.c_float), _p(inv, C.c_float), _p(off, C.c_float))
    return step, inv, off


PAIR_SELF, PAIR_REQUANT, PAIR_RAW = 0, 1, 2


def quant_metrics(x, y, outer: int, channels: int, inner: int, per_channel: bool, asym_u8: bool,
                  pair_mode: int, step, inv, offset, want_codes: bool = False, bits: int = 8):
    """-> dict(sse, sig, mse, sqnr_db[, codes])."""
    lib = _load()
    x = _f32(x).reshape(-1)
    yy = None if y is None else _f32(y).reshape(-1)
    if pair_mode != PAIR_SELF:
        assert yy is not None and yy.size == x.size
    step, inv, offset = _f32(step), _f32(inv), _f32(offset)
    codes = np.zeros(x.size, np.uint8) if want_codes else None
    out = [C.c_double(0.0) for _ in range(4)]
    lib.qv2o_quant_metrics_bits(int(bits), _p(x, C.c_float), _p(yy, C.c_float), outer, channels, inner,
                           int(per_channel), int(asym_u8), int(pair_mode),
                           _p(step, C.c_float), _p(inv, C.c_float), _p(offset, C.c_float),
                           _p(codes, C.c_uint8), *[C.byref(o) for o in out])
    res = dict(sse=out[0].value, sig=out[1].value, mse=out[2].value, sqnr_db=out[3].value)
    if want_codes:
        res["codes"] = codes if asym_u8 else codes.view(np.int8)
    return res


def cosine(x, y, outer: int, channels: int, inner: int, per_channel: bool, asym_u8: bool,
           pair_mode: int, step, inv, offset, bits: int = 8) -> float:
    """Cosine similarity between x and the tensor it is compared with (see quant_metrics)."""
    lib = _load()
    x = _f32(x).reshape(-1)
    yy = None if y is None else _f32(y).reshape(-1)
    step, inv, offset = _f32(step), _f32(inv), _f32(offset)
    return float(lib.qv2o_cosine_bits(int(bits), _p(x, C.c_float), _p(yy, C.c_float), outer, channels, inner,
                                 int(per_channel), int(asym_u8), int(pair_mode), _p(step, C.c_float),
                                 _p(inv, C.c_float), _p(offset, C.c_float)))


def fold_batchnorm(w, bias, gamma, beta, mean, var):
    """Eq. 10-12: -> (folded weights [C, K] float32, folded bias [C] float32)."""
    lib = _load()
    w = _f32(w)
    c, k = w.shape
    b = None if bias is None else _f32(bias)
    gamma, beta, mean, var = _f32(gamma), _f32(beta), _f32(mean), _f32(var)
    w_out = np.zeros((c, k), np.float32); b_out = np.zeros(c, np.float32)
    lib.qv2o_fold_batchnorm(_p(w, C.c_float), _p(b, C.c_float), _p(gamma, C.c_float), _p(beta, C.c_float),
                            _p(mean, C.c_float), _p(var, C.c_float), c, k, _p(w_out, C.c_float),
                            _p(b_out, C.c_float))
    return w_out, b_out


KL_BINS = 128


def kl_divergence(x, y, outer: int, channels: int, inner: int, per_channel: bool, asym_u8, pair_mode: int,
                  step, inv, offset, absmax: float, bits: int = 8):
    """-> (kl in nats, hist of |x| [128], hist of the compared tensor [128]); see qv2o_kl_bits."""
    lib = _load()
    x = _f32(x).reshape(-1)
    yy = None if y is None else _f32(y).reshape(-1)
    step, inv, offset = _f32(step), _f32(inv), _f32(offset)
    hp = np.zeros(KL_BINS, np.uint64); hq = np.zeros(KL_BINS, np.uint64)
    kl = lib.qv2o_kl_bits(int(bits), _p(x, C.c_float), _p(yy, C.c_float), outer, channels, inner,
                          int(per_channel), int(asym_u8), int(pair_mode), _p(step, C.c_float),
                          _p(inv, C.c_float), _p(offset, C.c_float), C.c_float(absmax),
                          _p(hp, C.c_uint64), _p(hq, C.c_uint64))
    return float(kl), hp, hq


def rank_layers(sqnr_w, mse_w, sqnr_a, mse_a, macs=None, pos=None, w_gain=2.0, a_gain=1.0,
                mse_factor=5.0, cap_db=200.0, select_mode=0, keep_count=0, rate_permyriad=0,
                outlier_order=0):
    """-> (order[n] uint32, keep_fp32[n] uint8, n_keep).  outlier_order 1 places the MSE outliers
    as Algorithm 2's pseudo-code does (each at the head when met: reverse layer order)."""
    lib = _load()
    f = lambda a: np.ascontiguousarray(a, dtype=np.float64)
    sqnr_w, mse_w, sqnr_a, mse_a = f(sqnr_w), f(mse_w), f(sqnr_a), f(mse_a)
    n = sqnr_w.size
    m = None if macs is None else np.ascontiguousarray(macs, dtype=np.uint64)
    ps = None if pos is None else f(pos)
    order = np.zeros(n, np.uint32); keep = np.zeros(n, np.uint8); nk = C.c_uint32(0)
    lib.qv2o_rank_ex(n, _p(sqnr_w, C.c_double), _p(mse_w, C.c_double), _p(sqnr_a, C.c_double),
                     _p(mse_a, C.c_double), _p(m, C.c_uint64), _p(ps, C.c_double),
                     w_gain, a_gain, mse_factor, cap_db, int(select_mode), int(keep_count),
                     int(rate_permyriad), int(outlier_order), _p(order, C.c_uint32), _p(keep, C.c_uint8),
                     C.byref(nk))
    return order, keep, int(nk.value)


NO_GROUP = 0xFFFFFFFF


def rank_layers_fused(sqnr_w, mse_w, sqnr_a, mse_a, fuse_group, macs=None, pos=None, w_gain=2.0,
                      a_gain=1.0, mse_factor=5.0, cap_db=200.0, select_mode=0, keep_count=0,
                      rate_permyriad=0, outlier_order=0):
    """rank_layers with fusion groups: -> (order, keep_fp32, n_keep).  fuse_group[i] is a group id
    or NO_GROUP; None means no groups at all."""
    lib = _load()
    f = lambda a: np.ascontiguousarray(a, dtype=np.float64)
    sqnr_w, mse_w, sqnr_a, mse_a = f(sqnr_w), f(mse_w), f(sqnr_a), f(mse_a)
    n = sqnr_w.size
    m = None if macs is None else np.ascontiguousarray(macs, dtype=np.uint64)
    ps = None if pos is None else f(pos)
    fg = None if fuse_group is None else np.ascontiguousarray(fuse_group, dtype=np.uint32)
    order = np.zeros(n, np.uint32); keep = np.zeros(n, np.uint8); nk = C.c_uint32(0)
    lib.qv2o_rank_fused_ex(n, _p(sqnr_w, C.c_double), _p(mse_w, C.c_double), _p(sqnr_a, C.c_double),
                           _p(mse_a, C.c_double), _p(m, C.c_uint64), _p(ps, C.c_double), _p(fg, C.c_uint32),
                           w_gain, a_gain, mse_factor, cap_db, int(select_mode), int(keep_count),
                           int(rate_permyriad), int(outlier_order), _p(order, C.c_uint32), _p(keep, C.c_uint8),
                           C.byref(nk))
    return order, keep, int(nk.value)


# --------------------------------------------------------------------------- per-tensor sweep
@dataclass
class TensorResult:
    gmin: np.ndarray
    gmax: np.ndarray
    gabsmax: np.ndarray
    nonfinite: int
    hist: Optional[np.ndarray]
    clip: np.float32
    step: np.ndarray
    inv: np.ndarray
    offset: np.ndarray
    sse: float
    sig: float
    mse: float
    sqnr_db: float
    codes: Optional[np.ndarray] = None
    ghist: Optional[np.ndarray] = None     # [groups][2048], per-group percentile calibration only
    gclip: Optional[np.ndarray] = None     # clip bound applied to each group


def calibrate_tensor(x, outer, channels, inner, per_channel, asym_u8, percentile=None, bits=8,
                     group_percentile=False):
    """Ranges, optional |x| histogram + percentile clip, then the quantization parameters.
    ``group_percentile`` (per-channel tensors only) takes one histogram and one clip per channel
    instead of one per tensor; the tensor-level clip is then the plain absmax and hist is None."""
    gmin, gmax, gabs, bad = ranges(x, outer, channels, inner, per_channel)
    A = np.float32(gabs.max()) if gabs.size else np.float32(0.0)
    hist, clip, ghist = None, A, None
    if percentile is not None and group_percentile and per_channel:
        ghist, gclip = group_histograms(x, outer, channels, inner, gabs, percentile)
        step, inv, off = qparams_gclip(asym_u8, gmin, gmax, gabs, gclip, bits)
        return gmin, gmax, gabs, bad, hist, clip, step, inv, off, ghist, gclip
    if percentile is not None:
        hist = histogram(x, float(A))
        clip = percentile_clip(hist, percentile, float(A))
    step, inv, off = qparams(asym_u8, gmin, gmax, gabs, None if percentile is None else float(clip), bits)
    return gmin, gmax, gabs, bad, hist, clip, step, inv, off, ghist, np.full(gabs.size, clip, np.float32)


def sweep_tensor(x, y, outer, channels, inner, per_channel, asym_u8, percentile=None,
                 pair_mode=None, want_codes=False, bits=8, group_percentile=False) -> TensorResult:
    """Calibrate on x, then measure: self mode when y is None, else the paired mode."""
    gmin, gmax, gabs, bad, hist, clip, step, inv, off, ghist, gclip = calibrate_tensor(
        x, outer, channels, inner, per_channel, asym_u8, percentile, bits, group_percentile)
    if pair_mode is None:
        pair_mode = PAIR_SELF if y is None else PAIR_REQUANT
    m = quant_metrics(x, y, outer, channels, inner, per_channel, asym_u8, pair_mode,
                      step, inv, off, want_codes, bits)
    return TensorResult(gmin, gmax, gabs, bad, hist, clip, step, inv, off,
                        m["sse"], m["sig"], m["mse"], m["sqnr_db"], m.get("codes"), ghist, gclip)


def sweep_tensors(jobs: Sequence[dict], threads: int = 1) -> List[TensorResult]:
    """Run sweep_tensor over independent tensors.  ``threads`` > 1 runs whole tensors side by
    side (the C calls release the GIL); each tensor is still swept by the serial code above."""
    if threads <= 1:
        return [sweep_tensor(**j) for j in jobs]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(lambda j: sweep_tensor(**j), jobs))
