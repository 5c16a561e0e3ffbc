"""qv2_quant_metrics_noalloc: the metrics pass for callers that are not allowed to allocate.

Some users of this library run it where cudaMalloc is forbidden -- a server that gave all device
memory to its own pool at start-up, a latency-critical loop in which an allocation would stall the
GPU, a host callback.  For them the library offers one entry point that needs no context and keeps
its partial sums in a fixed 1 MiB array inside the library image.  These tests call it through the
C ABI and compare it with the regular qv2_quant_metrics on the same inputs and parameters and,
independently, with the CPU oracle (the same 1e-5 / 1e-3 dB bars, so no two tolerances stack), twice
in a row (the array is shared between calls and still holds the previous call's data, so the
second call is the one that would expose stale state), and check that a tensor beyond the stated
limit is refused with QV2_ERR_SIZE instead of being launched.

The file name sorts last so that a run that stops at the first failure has already run every
other test.  It passes on its own in a fresh process and after the rest of the suite.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2501_07161_b200 as q
from paper_2501_07161_b200 import binding as B

pytestmark = pytest.mark.gpu

MSE_RTOL = 1e-5          # the same bars as the oracle parity tests
SQNR_ATOL_DB = 1e-3
TILE = 16384


def _gen(seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return g


def _cases():
    n = 5 * TILE + 1234
    x = torch.randn(n, generator=_gen(1), device="cuda")
    y = x + 0.02 * torch.randn(n, generator=_gen(2), device="cuda")
    w = torch.randn(96 * 1153, generator=_gen(3), device="cuda")            # short ragged rows
    wl = torch.randn(3 * 20000, generator=_gen(4), device="cuda")           # rows cut at row ends
    a = torch.randn(4 * 6 * 500, generator=_gen(5), device="cuda").clamp_min(0)
    s = torch.randn(5 * 37 * 9, generator=_gen(6), device="cuda")           # rows of nine elements
    s2 = s + 0.05 * torch.randn(5 * 37 * 9, generator=_gen(9), device="cuda")
    m = torch.randn(3 * 70 * 300, generator=_gen(10), device="cuda") + 0.7   # 54 rows per tile, three tiles and a tail
    m2 = m + 0.03 * torch.randn(3 * 70 * 300, generator=_gen(11), device="cuda")
    return [
        ("activation pair, asymmetric, offset != 0", x, y, (1, 1, n), B.PER_TENSOR, B.ASYM_U8, B.MINMAX, 0),
        ("activation pair, raw difference", x, y, (1, 1, n), B.PER_TENSOR, B.ASYM_U8, B.MINMAX, B.PAIR_RAW),
        ("weights, per channel, short rows", w, None, (1, 96, 1153), B.PER_CHANNEL, B.SYM_I8, B.ABSMAX, 0),
        ("weights, per channel, long rows", wl, None, (1, 3, 20000), B.PER_CHANNEL, B.SYM_I8, B.ABSMAX, 0),
        ("relu activation, per channel with batch, percentile", a, None, (4, 6, 500), B.PER_CHANNEL,
         B.ASYM_U8, B.PERCENTILE, 0),
        ("one element", x[:1].clone(), None, (1, 1, 1), B.PER_TENSOR, B.SYM_I8, B.ABSMAX, 0),
        ("rows shorter than a warp, per channel, pair", s, s2, (5, 37, 9), B.PER_CHANNEL, B.ASYM_U8, B.MINMAX, 0),
        ("rows shorter than a warp, weights", s, None, (1, 185, 9), B.PER_CHANNEL, B.SYM_I8, B.ABSMAX, 0),
        ("per channel, row count per tile not a multiple of eight", m, m2, (3, 70, 300), B.PER_CHANNEL,
         B.ASYM_U8, B.MINMAX, 0),
        ("integer zero point, per tensor", x + 0.4, y + 0.4, (1, 1, n), B.PER_TENSOR, B.ASYM_U8_ZP, B.MINMAX, 0),
        ("integer zero point, per channel", m, m2, (3, 70, 300), B.PER_CHANNEL, B.ASYM_U8_ZP, B.MINMAX, 0),
        ("4-bit symmetric weights", w, None, (1, 96, 1153), B.PER_CHANNEL, B.SYM_I8, B.ABSMAX, 4 << 8),
        ("4-bit affine activations", x, y, (1, 1, n), B.PER_TENSOR, B.ASYM_U8, B.MINMAX, 4 << 8),
    ]


def _oracle4(x, y, shape, gran, scheme, rng, flags, step, inv, offset):
    """The oracle's metrics for the parameters the call is given (the GPU calibration's bits, which the
    parity tests pin to the oracle's own)."""
    o, c, i = shape
    bits = ((flags >> 8) & 0xFF) or 8
    mode = oracle.PAIR_SELF if y is None else (oracle.PAIR_RAW if flags & B.PAIR_RAW else oracle.PAIR_REQUANT)
    r = oracle.quant_metrics(x.cpu().numpy(), None if y is None else y.cpu().numpy(), o, c, i,
                             gran == B.PER_CHANNEL, int(scheme), mode, step.cpu().numpy(), inv.cpu().numpy(),
                             offset.cpu().numpy(), bits=bits)
    return r["sse"], r["sig"], r["mse"], r["sqnr_db"]


def _close(got, ref, what):
    sse, sig, mse, sqnr = (float(v) for v in got)
    rsse, rsig, rmse, rsqnr = (float(v) for v in ref)
    assert abs(mse - rmse) <= MSE_RTOL * abs(rmse), f"{what}: mse {mse} vs {rmse}"
    assert abs(sse - rsse) <= MSE_RTOL * abs(rsse), f"{what}: sse {sse} vs {rsse}"
    assert abs(sig - rsig) <= MSE_RTOL * abs(rsig), f"{what}: sig {sig} vs {rsig}"
    if math.isinf(rsqnr):
        assert sqnr == rsqnr, what
    else:
        assert abs(sqnr - rsqnr) <= SQNR_ATOL_DB, f"{what}: sqnr {sqnr} vs {rsqnr}"


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    ctx = q.Context(0)
    try:
        for name, x, y, (o, c, i), gran, scheme, rng, flags in _cases():
            desc = q.make_desc(x, y, o, c, i, gran, scheme, rng, 0.999, flags)
            descs = q.desc_array([desc])
            cal = ctx.calibrate(descs)
            ref = ctx.quant_metrics(descs, cal.step, cal.inv, cal.offset)
            torch.cuda.synchronize()
            ref4 = (ref.sse[0], ref.sig[0], ref.mse[0], ref.sqnr_db[0])
            # the oracle calibrates to the same parameter bits, so both references see one quantizer
            oc = oracle.calibrate_tensor(x.cpu().numpy(), o, c, i, gran == B.PER_CHANNEL, int(scheme),
                                         0.999 if rng == B.PERCENTILE else None, ((flags >> 8) & 0xFF) or 8)
            assert np.array_equal(cal.step.cpu().numpy().view(np.uint32), oc[6].view(np.uint32)), name
            assert np.array_equal(cal.offset.cpu().numpy().view(np.uint32), oc[8].view(np.uint32)), name
            ora4 = _oracle4(x, y, (o, c, i), gran, scheme, rng, flags, cal.step, cal.inv, cal.offset)
            for call in (1, 2):
                out = torch.full((4,), float("nan"), dtype=torch.float64, device="cuda")
                st = B.quant_metrics_noalloc(desc, cal.step, cal.inv, cal.offset, out)
                assert st == 0, f"{name}: status {st}"
                torch.cuda.synchronize()
                _close(out.tolist(), ref4, f"{name} (call {call}, against qv2_quant_metrics)")
                _close(out.tolist(), ora4, f"{name} (call {call}, against the oracle)")
    finally:
        ctx.close()


def test_noalloc_after_a_larger_tensor_ignores_stale_partials():
    """A big call fills many slots; the small call that follows must not read them."""
    ctx = q.Context(0)
    try:
        big = torch.randn(40 * TILE, generator=_gen(7), device="cuda") * 100.0
        small = torch.randn(TILE // 2 + 3, generator=_gen(8), device="cuda") * 0.01
        for t in (big, small):
            desc = q.make_desc(t, None, 1, 1, t.numel(), B.PER_TENSOR, B.SYM_I8)
            descs = q.desc_array([desc])
            cal = ctx.calibrate(descs)
            ref = ctx.quant_metrics(descs, cal.step, cal.inv, cal.offset)
            out = torch.zeros(4, dtype=torch.float64, device="cuda")
            assert B.quant_metrics_noalloc(desc, cal.step, cal.inv, cal.offset, out) == 0
            torch.cuda.synchronize()
            _close(out.tolist(), (ref.sse[0], ref.sig[0], ref.mse[0], ref.sqnr_db[0]), f"n={t.numel()}")
            _close(out.tolist(), _oracle4(t, None, (1, 1, t.numel()), B.PER_TENSOR, B.SYM_I8, B.ABSMAX, 0,
                                          cal.step, cal.inv, cal.offset), f"n={t.numel()} against the oracle")
    finally:
        ctx.close()


def test_noalloc_rejects_sizes_beyond_the_fixed_scratch():
    x = torch.zeros(16, device="cuda")
    p = torch.ones(1, device="cuda")
    out = torch.zeros(4, dtype=torch.float64, device="cuda")
    too_big = q.make_desc(x, None, 1, 1, B.NOALLOC_MAX_ELEMS + 1, B.PER_TENSOR, B.SYM_I8)
    assert B.quant_metrics_noalloc(too_big, p, p, p, out) == -4          # QV2_ERR_SIZE
    assert b"SIZE" in q.lib().qv2_status_string(-4)
    # ragged long rows: fewer elements than the limit but more tiles than the array has room for
    ragged = q.make_desc(x, None, 1, 8000, 16385, B.PER_CHANNEL, B.SYM_I8)
    assert 8000 * 16385 <= B.NOALLOC_MAX_ELEMS
    assert B.quant_metrics_noalloc(ragged, p, p, p, out) == -4
    with_codes = q.make_desc(x, None, 1, 1, 16, B.PER_TENSOR, B.SYM_I8, flags=B.STORE_CODES)
    assert B.quant_metrics_noalloc(with_codes, p, p, p, out) == -1       # QV2_ERR_ARG
    torch.cuda.synchronize()
    assert out.tolist() == [0.0, 0.0, 0.0, 0.0]                          # nothing was launched
