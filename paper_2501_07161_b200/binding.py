"""Thin ctypes binding of libqv2.so: the same entry points as include/qv2.h, argument marshalling
only.  torch supplies device memory and the stream; every step of the sweep runs in the library's
CUDA kernels.  There is no CPU fallback: if the library cannot be built or loaded, importing
``lib()`` raises."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

from . import build as _build

PER_TENSOR, PER_CHANNEL = 0, 1
SYM_I8, ASYM_U8, ASYM_U8_ZP = 0, 1, 2
ABSMAX, MINMAX, PERCENTILE, PERCENTILE_GROUP = 0, 1, 2, 3
PAIR_REQUANT, PAIR_RAW, STORE_CODES = 0, 1, 2
BY_COUNT, BY_BOPS_RATE = 0, 1
OUTLIERS_BY_SEVERITY, OUTLIERS_LITERAL = 0, 1
SCHEDULE_PHASE_MAJOR, SCHEDULE_L2_CHUNKED, SCHEDULE_AUTO = 0, 1, 2
FOLD_AUTO, FOLD_FUSED, FOLD_SEPARATE = 0, 1, 2
IN_F32, IN_F16, IN_BF16 = 0, 1 << 16, 2 << 16
_DTYPE_FLAG = {torch.float32: IN_F32, torch.float16: IN_F16, torch.bfloat16: IN_BF16}
HIST_BINS = 2048
OK = 0

EXPORTS = ["qv2_create", "qv2_destroy", "qv2_status_string", "qv2_last_cuda_error",
           "qv2_launch_count", "qv2_group_count", "qv2_calibrate", "qv2_quant_metrics",
           "qv2_rank_layers", "qv2_sweep_model", "qv2_sweep_model_host", "qv2_staging_bytes",
           "qv2_debug_plan_tiles", "qv2_quant_metrics_noalloc", "qv2_quant_metrics_ex", "qv2_rank_layers_ex", "qv2_kl_divergence", "qv2_fold_batchnorm", "qv2_sweep_graph_create", "qv2_sweep_graph_launch",
           "qv2_sweep_graph_destroy", "qv2_check_nonfinite", "qv2_calibrate_ex", "qv2_group_hist_count",
           "qv2_sync_count", "qv2_set_schedule", "qv2_stage_count", "qv2_set_fold_mode",
           "qv2_set_phase_timing", "qv2_calibrate_phase_ms", "qv2_set_dependent_launch"]
KL_BINS = 128
NO_GROUP = 0xFFFFFFFF
NOALLOC_MAX_ELEMS = 1 << 27


class TensorDesc(C.Structure):
    _fields_ = [("x", C.c_void_p), ("y", C.c_void_p),
                ("outer", C.c_uint64), ("channels", C.c_uint64), ("inner", C.c_uint64),
                ("granularity", C.c_uint32), ("scheme", C.c_uint32), ("range", C.c_uint32),
                ("flags", C.c_uint32), ("percentile", C.c_double)]


class RankCfg(C.Structure):
    _fields_ = [("w_gain", C.c_double), ("a_gain", C.c_double), ("mse_factor", C.c_double),
                ("sqnr_cap_db", C.c_double), ("select_mode", C.c_uint32),
                ("keep_count", C.c_uint32), ("rate_permyriad", C.c_uint32),
                ("outlier_order", C.c_uint32)]


class SweepBuffers(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("gmin", "gmax", "gabsmax", "step", "inv", "offset", "hist", "clip", "nonfinite",
                 "sse", "sig", "mse", "sqnr_db", "order", "keep_fp32", "n_keep")]


class HostResults(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("mse", "sqnr_db", "nonfinite", "order", "keep_fp32", "n_keep")]


_lib = None


def lib() -> C.CDLL:
    """Builds (if stale) and loads libqv2.so; raises when that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    L = C.CDLL(path)
    vp, u32, u64, i32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int
    dp = C.POINTER(TensorDesc)
    L.qv2_create.argtypes = [C.POINTER(vp), i32, vp]; L.qv2_create.restype = i32
    L.qv2_destroy.argtypes = [vp]; L.qv2_destroy.restype = i32
    L.qv2_status_string.argtypes = [i32]; L.qv2_status_string.restype = C.c_char_p
    L.qv2_last_cuda_error.argtypes = [vp]; L.qv2_last_cuda_error.restype = i32
    L.qv2_launch_count.argtypes = [vp]; L.qv2_launch_count.restype = u64
    L.qv2_sync_count.argtypes = [vp]; L.qv2_sync_count.restype = u64
    L.qv2_set_schedule.argtypes = [vp, u32, u64]; L.qv2_set_schedule.restype = i32
    L.qv2_stage_count.argtypes = [vp]; L.qv2_stage_count.restype = u32
    L.qv2_set_fold_mode.argtypes = [vp, u32]; L.qv2_set_fold_mode.restype = i32
    L.qv2_set_dependent_launch.argtypes = [vp, i32]; L.qv2_set_dependent_launch.restype = i32
    L.qv2_set_phase_timing.argtypes = [vp, i32]; L.qv2_set_phase_timing.restype = i32
    L.qv2_calibrate_phase_ms.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_float)]
    L.qv2_calibrate_phase_ms.restype = i32
    L.qv2_group_count.argtypes = [dp, u32]; L.qv2_group_count.restype = u64
    L.qv2_calibrate.argtypes = [vp, dp, u32] + [vp] * 9; L.qv2_calibrate.restype = i32
    L.qv2_calibrate_ex.argtypes = [vp, dp, u32] + [vp] * 11; L.qv2_calibrate_ex.restype = i32
    L.qv2_group_hist_count.argtypes = [dp, u32]; L.qv2_group_hist_count.restype = C.c_uint64
    L.qv2_quant_metrics.argtypes = [vp, dp, u32, vp, vp, vp, C.POINTER(vp), vp, vp, vp, vp]
    L.qv2_quant_metrics.restype = i32
    L.qv2_quant_metrics_ex.argtypes = [vp, dp, u32, vp, vp, vp, C.POINTER(vp), vp, vp, vp, vp, vp]
    L.qv2_quant_metrics_ex.restype = i32
    L.qv2_rank_layers.argtypes = [vp, u32, vp, vp, vp, vp, vp, vp, C.POINTER(RankCfg), vp, vp, vp]
    L.qv2_rank_layers.restype = i32
    L.qv2_kl_divergence.argtypes = [vp, dp, u32, vp, vp, vp, vp, vp, vp]
    L.qv2_kl_divergence.restype = i32
    L.qv2_check_nonfinite.argtypes = [vp, vp, u32, C.POINTER(u32)]; L.qv2_check_nonfinite.restype = i32
    L.qv2_sweep_graph_create.argtypes = [vp, dp, u32, u32, vp, vp, C.POINTER(RankCfg), C.POINTER(SweepBuffers),
                                         C.POINTER(vp)]
    L.qv2_sweep_graph_create.restype = i32
    L.qv2_sweep_graph_launch.argtypes = [vp]; L.qv2_sweep_graph_launch.restype = i32
    L.qv2_sweep_graph_destroy.argtypes = [vp]; L.qv2_sweep_graph_destroy.restype = i32
    L.qv2_fold_batchnorm.argtypes = [vp, vp, vp, vp, vp, vp, vp, u64, u64, vp, vp]
    L.qv2_fold_batchnorm.restype = i32
    L.qv2_rank_layers_ex.argtypes = [vp, u32, vp, vp, vp, vp, vp, vp, vp, C.POINTER(RankCfg), vp, vp, vp]
    L.qv2_rank_layers_ex.restype = i32
    L.qv2_sweep_model.argtypes = [vp, dp, u32, u32, vp, vp, C.POINTER(RankCfg),
                                  C.POINTER(SweepBuffers)]
    L.qv2_sweep_model.restype = i32
    L.qv2_sweep_model_host.argtypes = [vp, dp, u32, u32, vp, vp, C.POINTER(RankCfg), vp, u64,
                                       C.POINTER(SweepBuffers), C.POINTER(HostResults)]
    L.qv2_sweep_model_host.restype = i32
    L.qv2_staging_bytes.argtypes = [dp, u32, u32]; L.qv2_staging_bytes.restype = u64
    L.qv2_debug_plan_tiles.argtypes = [dp, u32, vp, u64]; L.qv2_debug_plan_tiles.restype = C.c_int64
    L.qv2_quant_metrics_noalloc.argtypes = [i32, vp, dp, vp, vp, vp, vp]
    L.qv2_quant_metrics_noalloc.restype = i32
    _lib = L
    return L


class Qv2Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().qv2_status_string(status).decode()} ({status})")


def _check(status: int, where: str):
    if status != OK:
        raise Qv2Error(status, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def make_desc(x: Optional[torch.Tensor], y: Optional[torch.Tensor], outer: int, channels: int,
              inner: int, granularity: int, scheme: int, range_mode: int = ABSMAX,
              percentile: float = 0.0, flags: int = 0, bits: int = 8) -> TensorDesc:
    d = TensorDesc()
    if x is not None:                     # the element type travels in the flags
        if x.dtype not in _DTYPE_FLAG or (y is not None and y.dtype != x.dtype):
            raise TypeError("x and y must both be float32, float16 or bfloat16")
        flags |= _DTYPE_FLAG[x.dtype]
    d.x = _ptr(x) if x is not None and x.numel() else None
    d.y = _ptr(y) if y is not None and y.numel() else None
    if y is not None and not y.numel():
        d.y = None
    d.outer, d.channels, d.inner = outer, channels, inner
    d.granularity, d.scheme, d.range, d.flags = granularity, scheme, range_mode, flags | (0 if bits == 8 else bits << 8)
    d.percentile = percentile
    return d


def desc_array(descs: Sequence[TensorDesc]):
    arr = (TensorDesc * len(descs))()
    for i, d in enumerate(descs):
        arr[i] = d
    return arr


def default_rank_cfg(select_mode=BY_COUNT, keep_count=0, rate_permyriad=0, w_gain=2.0, a_gain=1.0,
                     mse_factor=5.0, sqnr_cap_db=200.0, outlier_order=OUTLIERS_BY_SEVERITY) -> RankCfg:
    return RankCfg(w_gain, a_gain, mse_factor, sqnr_cap_db, select_mode, keep_count, rate_permyriad,
                   outlier_order)


@dataclass
class CalibOut:
    gmin: torch.Tensor
    gmax: torch.Tensor
    gabsmax: torch.Tensor
    hist: Optional[torch.Tensor]
    clip: torch.Tensor
    step: torch.Tensor
    inv: torch.Tensor
    offset: torch.Tensor
    nonfinite: torch.Tensor
    group_hist: Optional[torch.Tensor] = None     # [qv2_group_hist_count][2048]
    group_clip: Optional[torch.Tensor] = None     # per group


@dataclass
class MetricsOut:
    sse: torch.Tensor
    sig: torch.Tensor
    mse: torch.Tensor
    sqnr_db: torch.Tensor
    codes: Optional[List[Optional[torch.Tensor]]] = None
    cosine: Optional[torch.Tensor] = None


class Context:
    """One qv2_ctx bound to a device and to torch's current stream on it."""

    def __init__(self, device: int = 0, stream: Optional[torch.cuda.Stream] = None):
        self._h = C.c_void_p()
        self.device = torch.device("cuda", device)
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        self.stream = s
        self._graphs = []          # captured passes must be destroyed before their context
        _check(lib().qv2_create(C.byref(self._h), device, C.c_void_p(s.cuda_stream)), "qv2_create")

    def close(self):
        for g in getattr(self, "_graphs", []):
            g.close()
        self._graphs = []
        if self._h:
            lib().qv2_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def launches(self) -> int:
        return int(lib().qv2_launch_count(self._h))

    @property
    def syncs(self) -> int:
        return int(lib().qv2_sync_count(self._h))

    @property
    def stages(self) -> int:
        return int(lib().qv2_stage_count(self._h))

    def set_schedule(self, schedule: int, chunk_bytes: int = 0):
        _check(lib().qv2_set_schedule(self._h, schedule, chunk_bytes), "qv2_set_schedule")

    def set_fold_mode(self, mode: int):
        _check(lib().qv2_set_fold_mode(self._h, mode), "qv2_set_fold_mode")

    def set_dependent_launch(self, on: bool):
        _check(lib().qv2_set_dependent_launch(self._h, int(on)), "qv2_set_dependent_launch")

    def set_phase_timing(self, on: bool):
        _check(lib().qv2_set_phase_timing(self._h, int(on)), "qv2_set_phase_timing")

    def calibrate_phase_ms(self):
        """(range_ms, hist_ms) of the most recent timed qv2_calibrate; synchronises."""
        r, h = C.c_float(0.0), C.c_float(0.0)
        _check(lib().qv2_calibrate_phase_ms(self._h, C.byref(r), C.byref(h)), "qv2_calibrate_phase_ms")
        return float(r.value), float(h.value)

    def last_cuda_error(self) -> int:
        return int(lib().qv2_last_cuda_error(self._h))

    # -- allocation helpers (torch is only the allocator) ---------------------------------
    def _empty(self, n, dtype):
        return torch.empty(max(int(n), 1), dtype=dtype, device=self.device)

    def alloc_sweep_buffers(self, descs, n_layers: int, want_hist: bool = True):
        n = len(descs)
        g = int(lib().qv2_group_count(descs, n))
        t = {k: self._empty(g, torch.float32) for k in ("gmin", "gmax", "gabsmax", "step", "inv", "offset")}
        t["hist"] = self._empty(n * HIST_BINS, torch.int64) if want_hist else None
        t["clip"] = self._empty(n, torch.float32)
        t["nonfinite"] = self._empty(n, torch.int64)
        for k in ("sse", "sig", "mse", "sqnr_db"):
            t[k] = self._empty(n, torch.float64)
        t["order"] = self._empty(n_layers, torch.int32)
        t["keep_fp32"] = self._empty(n_layers, torch.uint8)
        t["n_keep"] = self._empty(1, torch.int32)
        sb = SweepBuffers(**{k: _ptr(v) for k, v in t.items()})
        return sb, t

    # -- the three calls of the contract ---------------------------------------------------
    def calibrate(self, descs, want_hist: bool = True, want_group: bool = False) -> CalibOut:
        """qv2_calibrate; with want_group, qv2_calibrate_ex returning the per-group histograms and clips."""
        n = len(descs)
        g = int(lib().qv2_group_count(descs, n))
        f = lambda k: self._empty(k, torch.float32)
        out = CalibOut(f(g), f(g), f(g), self._empty(n * HIST_BINS, torch.int64) if want_hist else None,
                       f(n), f(g), f(g), f(g), self._empty(n, torch.int64))
        if want_group:
            gh = int(lib().qv2_group_hist_count(descs, n))
            out.group_hist = self._empty(gh * HIST_BINS, torch.int64)
            out.group_clip = f(g)
            _check(lib().qv2_calibrate_ex(self._h, descs, n, _ptr(out.gmin), _ptr(out.gmax), _ptr(out.gabsmax),
                                          _ptr(out.hist), _ptr(out.clip), _ptr(out.step), _ptr(out.inv),
                                          _ptr(out.offset), _ptr(out.nonfinite), _ptr(out.group_hist),
                                          _ptr(out.group_clip)), "qv2_calibrate_ex")
            return out
        _check(lib().qv2_calibrate(self._h, descs, n, _ptr(out.gmin), _ptr(out.gmax), _ptr(out.gabsmax),
                                   _ptr(out.hist), _ptr(out.clip), _ptr(out.step), _ptr(out.inv),
                                   _ptr(out.offset), _ptr(out.nonfinite)), "qv2_calibrate")
        return out

    def quant_metrics(self, descs, step, inv, offset, codes: Optional[Sequence[Optional[torch.Tensor]]] = None,
                      want_cosine: bool = False) -> MetricsOut:
        n = len(descs)
        d = lambda: self._empty(n, torch.float64)
        out = MetricsOut(d(), d(), d(), d(), list(codes) if codes is not None else None)
        cp = None
        if codes is not None:
            cp = (C.c_void_p * n)(*[_ptr(c) for c in codes])
        if want_cosine:
            out.cosine = d()
            _check(lib().qv2_quant_metrics_ex(self._h, descs, n, _ptr(step), _ptr(inv), _ptr(offset), cp,
                                              _ptr(out.sse), _ptr(out.sig), _ptr(out.mse), _ptr(out.sqnr_db),
                                              _ptr(out.cosine)), "qv2_quant_metrics_ex")
            return out
        _check(lib().qv2_quant_metrics(self._h, descs, n, _ptr(step), _ptr(inv), _ptr(offset), cp,
                                       _ptr(out.sse), _ptr(out.sig), _ptr(out.mse), _ptr(out.sqnr_db)),
               "qv2_quant_metrics")
        return out

    def check_nonfinite(self, nonfinite: torch.Tensor):
        """-> (status, index of the first tensor with NaN/Inf or None); synchronises the stream."""
        bad = C.c_uint32(0xFFFFFFFF)
        st = int(lib().qv2_check_nonfinite(self._h, _ptr(nonfinite), nonfinite.numel(), C.byref(bad)))
        if st not in (OK, -5):
            raise Qv2Error(st, "qv2_check_nonfinite")
        return st, (int(bad.value) if st == -5 else None)

    def fold_batchnorm(self, w, bias, gamma, beta, mean, var, inplace: bool = False):
        """Eq. 10-12: -> (folded weights [C, K], folded bias [C]); inplace overwrites w."""
        c, k = w.shape
        w_out = w if inplace else torch.empty_like(w)
        b_out = self._empty(c, torch.float32)
        _check(lib().qv2_fold_batchnorm(self._h, _ptr(w), _ptr(bias), _ptr(gamma), _ptr(beta), _ptr(mean),
                                        _ptr(var), c, k, _ptr(w_out), _ptr(b_out)), "qv2_fold_batchnorm")
        return w_out, b_out[:c]

    def kl_divergence(self, descs, step, inv, offset, gabsmax, want_hists: bool = True):
        """-> (kl float64[n], hists int64[n, 2, 128] or None)."""
        n = len(descs)
        kl = self._empty(n, torch.float64)
        h = self._empty(n * 2 * KL_BINS, torch.int64) if want_hists else None
        _check(lib().qv2_kl_divergence(self._h, descs, n, _ptr(step), _ptr(inv), _ptr(offset), _ptr(gabsmax),
                                       _ptr(kl), _ptr(h)), "qv2_kl_divergence")
        return kl, (None if h is None else h.view(n, 2, KL_BINS))

    def rank_layers(self, sqnr_w, mse_w, sqnr_a, mse_a, macs=None, pos=None, cfg: Optional[RankCfg] = None,
                    fuse_group: Optional[torch.Tensor] = None):
        n = sqnr_w.numel()
        cfg = cfg or default_rank_cfg()
        order = self._empty(n, torch.int32)
        keep = self._empty(n, torch.uint8)
        nk = self._empty(1, torch.int32)
        if fuse_group is not None:
            _check(lib().qv2_rank_layers_ex(self._h, n, _ptr(sqnr_w), _ptr(mse_w), _ptr(sqnr_a), _ptr(mse_a),
                                            _ptr(macs), _ptr(pos), _ptr(fuse_group), C.byref(cfg),
                                            _ptr(order), _ptr(keep), _ptr(nk)), "qv2_rank_layers_ex")
            return order, keep, nk
        _check(lib().qv2_rank_layers(self._h, n, _ptr(sqnr_w), _ptr(mse_w), _ptr(sqnr_a), _ptr(mse_a),
                                     _ptr(macs), _ptr(pos), C.byref(cfg), _ptr(order), _ptr(keep),
                                     _ptr(nk)), "qv2_rank_layers")
        return order, keep, nk

    def sweep_model(self, descs, n_layers: int, macs, pos, cfg: RankCfg, bufs: SweepBuffers):
        _check(lib().qv2_sweep_model(self._h, descs, len(descs), n_layers, _ptr(macs), _ptr(pos),
                                     C.byref(cfg), C.byref(bufs)), "qv2_sweep_model")

    def sweep_graph(self, descs, n_layers: int, macs, pos, cfg: RankCfg, bufs: SweepBuffers) -> "SweepGraph":
        """Captures the pass once (the context must be on a non-default stream)."""
        h = C.c_void_p()
        _check(lib().qv2_sweep_graph_create(self._h, descs, len(descs), n_layers, _ptr(macs), _ptr(pos),
                                            C.byref(cfg), C.byref(bufs), C.byref(h)), "qv2_sweep_graph_create")
        g = SweepGraph(h, (descs, macs, pos, cfg, bufs))
        self._graphs.append(g)
        return g

    def sweep_model_host(self, host_descs, n_layers: int, macs_host, pos_host, cfg: RankCfg,
                         staging: torch.Tensor, bufs: SweepBuffers, out: HostResults) -> int:
        """Returns the status (OK or ERR_NONFINITE); other errors raise."""
        st = lib().qv2_sweep_model_host(self._h, host_descs, len(host_descs), n_layers,
                                        _ptr(macs_host), _ptr(pos_host), C.byref(cfg),
                                        _ptr(staging), staging.numel() * staging.element_size(),
                                        C.byref(bufs), C.byref(out))
        if st not in (OK, -5):
            raise Qv2Error(st, "qv2_sweep_model_host")
        return st


def quant_metrics_noalloc(desc: TensorDesc, step: torch.Tensor, inv: torch.Tensor, offset: torch.Tensor,
                          result4: torch.Tensor, device: int = 0,
                          stream: Optional[torch.cuda.Stream] = None) -> int:
    """qv2_quant_metrics_noalloc for one tensor: no context, no allocation inside the library.
    `result4` is a caller-owned float64[4] device tensor that receives {sse, sig, mse, sqnr_db}.
    Returns the status instead of raising so that callers can test the size limit."""
    s = stream if stream is not None else torch.cuda.current_stream(device)
    arr = (TensorDesc * 1)(desc)
    return int(lib().qv2_quant_metrics_noalloc(device, C.c_void_p(s.cuda_stream), arr, _ptr(step),
                                               _ptr(inv), _ptr(offset), _ptr(result4)))


class SweepGraph:
    """A captured pass; launch() replays it on the owning context's stream."""

    def __init__(self, handle, keepalive):
        self._h = handle
        self._keep = keepalive

    def launch(self):
        _check(lib().qv2_sweep_graph_launch(self._h), "qv2_sweep_graph_launch")

    def close(self):
        if self._h:
            lib().qv2_sweep_graph_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def staging_bytes(descs, n_layers: int) -> int:
    return int(lib().qv2_staging_bytes(descs, len(descs), n_layers))


def plan_tiles(descs):
    """Host-only: the tiles the kernels would walk, as a list of (tensor, begin, count, kind)."""
    import numpy as np
    n = len(descs)
    cnt = int(lib().qv2_debug_plan_tiles(descs, n, None, 0))
    if cnt < 0:
        raise Qv2Error(cnt, "qv2_debug_plan_tiles")
    buf = np.zeros((max(cnt, 1), 4), np.uint64)
    lib().qv2_debug_plan_tiles(descs, n, buf.ctypes.data, cnt)
    return [tuple(int(v) for v in row) for row in buf[:cnt]]
