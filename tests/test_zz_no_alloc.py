"""qv2_quant_metrics_noalloc: the metrics pass for callers that are not allowed to allocate.

Some users of this library run it where cudaMalloc is forbidden -- a server that gave all device
memory to its own pool at start-up, a latency-critical loop in which an allocation would stall the
GPU, a host callback.  For them the library offers one entry point that needs no context and keeps
its partial sums in a fixed 1 MiB array inside the library image.  These tests call it through the
C ABI and compare it with the regular qv2_quant_metrics on the same inputs and parameters, twice
in a row (the array is shared between calls and still holds the previous call's data, so the
second call is the one that would expose stale state), and check that a tensor beyond the stated
limit is refused with QV2_ERR_SIZE instead of being launched.

The file name sorts last so that a run that stops at the first failure has already run every
other test.  It passes on its own in a fresh process and after the rest of the suite.
"""
import math

import pytest
import torch

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
    return [
        ("activation pair, asymmetric, offset != 0", x, y, (1, 1, n), B.PER_TENSOR, B.ASYM_U8, B.MINMAX, 0),
        ("activation pair, raw difference", x, y, (1, 1, n), B.PER_TENSOR, B.ASYM_U8, B.MINMAX, B.PAIR_RAW),
        ("weights, per channel, short rows", w, None, (1, 96, 1153), B.PER_CHANNEL, B.SYM_I8, B.ABSMAX, 0),
        ("weights, per channel, long rows", wl, None, (1, 3, 20000), B.PER_CHANNEL, B.SYM_I8, B.ABSMAX, 0),
        ("relu activation, per channel with batch, percentile", a, None, (4, 6, 500), B.PER_CHANNEL,
         B.ASYM_U8, B.PERCENTILE, 0),
        ("one element", x[:1].clone(), None, (1, 1, 1), B.PER_TENSOR, B.SYM_I8, B.ABSMAX, 0),
    ]


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
            for call in (1, 2):
                out = torch.full((4,), float("nan"), dtype=torch.float64, device="cuda")
                st = B.quant_metrics_noalloc(desc, cal.step, cal.inv, cal.offset, out)
                assert st == 0, f"{name}: status {st}"
                torch.cuda.synchronize()
                _close(out.tolist(), ref4, f"{name} (call {call})")
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
