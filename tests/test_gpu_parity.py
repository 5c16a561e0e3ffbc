"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded
inputs, element by element.  Sizes span several 16384-element tiles and ragged tails; edge cases
cover empty, tiny, misaligned, constant, non-finite and on-grid tensors."""
import math

import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2501_07161_b200 as q
from parity import Spec, assert_metric_close, check_specs

pytestmark = pytest.mark.gpu

TILE = 16384


@pytest.fixture(scope="module", params=["fold-separate", "fold-fused"])
def ctx(request):
    """Every test runs twice: with the separate fold kernels (the default) and with the fold inside
    the streaming kernels."""
    c = q.Context(0)
    if request.param == "fold-fused":
        c.set_fold_mode(q.FOLD_FUSED)
    yield c
    c.close()


def _g(seed):
    g = torch.Generator()
    g.manual_seed(seed)
    return g


def randn(n, seed, scale=1.0):
    return torch.randn(n, generator=_g(seed)) * scale


# ------------------------------------------------------------------------ per-tensor, self mode
@pytest.mark.parametrize("n", [1, 2, 3, 5, 31, 1000, TILE - 1, TILE, TILE + 1, 3 * TILE + 777, 20 * TILE + 13])
@pytest.mark.parametrize("asym", [False, True])
def test_per_tensor_self_sizes(ctx, n, asym):
    check_specs(ctx, [Spec(randn(n, n), 1, 1, n, asym=asym)])


@pytest.mark.parametrize("mis", [1, 2, 3])
def test_misaligned_base_pointer(ctx, mis):
    n = 2 * TILE + 5
    check_specs(ctx, [Spec(randn(n, 7), 1, 1, n), Spec(randn(n, 8).abs(), 1, 1, n, asym=True)],
                misalign_x=mis)


def test_relu_activation_has_zero_offset_and_percentile(ctx):
    n = 5 * TILE + 99
    x = randn(n, 11).clamp_min(0)
    check_specs(ctx, [Spec(x, 1, 1, n, asym=True, percentile=0.9999),
                      Spec(x, 1, 1, n, asym=True, percentile=0.99),
                      Spec(randn(n, 12), 1, 1, n, asym=True, percentile=0.999),
                      Spec(randn(n, 13), 1, 1, n, asym=False, percentile=0.999)])


# --------------------------------------------------------------------------------- per channel
@pytest.mark.parametrize("cout,k", [(7, 1), (960, 9), (64, 27), (96, 147), (130, 576), (33, 1153),
                                    (9, 4095), (5, 4096), (5, 4097), (3, 25088), (2, 2 * TILE + 3)])
def test_per_channel_weights(ctx, cout, k):
    w = randn(cout * k, cout + k) * torch.exp(randn(cout, 3)).repeat_interleave(k)
    check_specs(ctx, [Spec(w, 1, cout, k, per_channel=True),
                      Spec(w, 1, cout, k, per_channel=True, asym=True)])


@pytest.mark.parametrize("o,c,i", [(3, 5, 100), (2, 3, 5000), (4, 2, TILE + 7), (17, 4, 49), (2, 1, 9)])
def test_per_channel_with_outer_dimension(ctx, o, c, i):
    x = randn(o * c * i, o + c + i) * torch.exp(randn(c, 5)).repeat_interleave(i).repeat(o)
    y = x + 0.01 * randn(x.numel(), 99)
    check_specs(ctx, [Spec(x, o, c, i, per_channel=True, asym=True, y=y),
                      Spec(x, o, c, i, per_channel=True, asym=False),
                      Spec(x, o, c, i, per_channel=True, asym=True, percentile=0.995)])


# ----------------------------------------------------------------------------------- pair modes
@pytest.mark.parametrize("mx,my", [(0, 0), (1, 1), (0, 2), (3, 1)])
def test_pair_modes_and_mixed_alignment(ctx, mx, my):
    n = 4 * TILE + 321
    x = randn(n, 21)
    y = x + 0.02 * randn(n, 22)
    xr = x.clamp_min(0)
    yr = xr + 0.02 * randn(n, 23)
    check_specs(ctx, [Spec(x, 1, 1, n, asym=True, y=y),               # offset != 0
                      Spec(xr, 1, 1, n, asym=True, y=yr),             # offset == 0
                      Spec(x, 1, 1, n, asym=True, y=y, raw=True),
                      Spec(x, 1, 1, n, asym=False, y=y),
                      Spec(x[: 8 * (n // 8)], 2, 4, n // 8, per_channel=True, asym=True,
                           y=y[: 8 * (n // 8)])],
                misalign_x=mx, misalign_y=my)


# ----------------------------------------------------------------------------------- edge cases
def test_empty_constant_and_zero_tensors_in_one_batch(ctx):
    specs = [Spec(torch.zeros(0), 0, 3, 5, per_channel=True),
             Spec(randn(100, 1), 1, 1, 100),
             Spec(torch.zeros(0), 1, 1, 0, asym=True, percentile=0.99),
             Spec(torch.zeros(1000), 1, 1, 1000, asym=True, percentile=0.99),
             Spec(torch.full((1000,), 2.5), 1, 1, 1000, asym=True),
             Spec(torch.full((1000,), -2.5), 1, 4, 250, per_channel=True),
             Spec(-torch.zeros(8), 1, 1, 8)]
    cal, met = check_specs(ctx, specs)
    assert float(met.sqnr_db[0]) == math.inf and float(met.mse[0]) == 0.0


def test_on_grid_tensor_zero_error(ctx):
    d = 2.0 ** -7
    k = torch.arange(-127, 128, dtype=torch.float32).repeat(300)
    cal, met = check_specs(ctx, [Spec(k * d, 1, 1, k.numel())])
    assert float(met.sse[0]) == 0.0 and float(met.sqnr_db[0]) == math.inf


def test_exact_ties_round_to_even(ctx):
    d = 2.0 ** -7
    k = torch.arange(-126, 126, dtype=torch.float32)
    x = torch.cat([(k + 0.5) * d, torch.tensor([127 * d, -127 * d])]).repeat(70)
    check_specs(ctx, [Spec(x, 1, 1, x.numel())])


def test_nonfinite_inputs_are_counted_and_excluded(ctx):
    n = 3 * TILE + 50
    x = randn(n, 31)
    x[0] = float("nan"); x[5] = float("inf"); x[TILE + 3] = float("-inf"); x[n - 1] = float("nan")
    x[2 * TILE + 17] = float("inf")
    w = randn(40 * 300, 32)
    w[7 * 300 + 5] = float("nan"); w[39 * 300 + 299] = float("inf")
    cal, _ = check_specs(ctx, [Spec(x, 1, 1, n, asym=True, percentile=0.99),
                               Spec(w, 1, 40, 300, per_channel=True),
                               Spec(randn(1000, 33), 1, 1, 1000)], check_codes=False)
    assert cal.nonfinite.tolist() == [5, 2, 0]
    assert ctx.check_nonfinite(cal.nonfinite) == (-5, 0)
    assert ctx.check_nonfinite(cal.nonfinite[2:]) == (0, None)


def test_extreme_magnitudes(ctx):
    """Squares are accumulated in binary32, so magnitudes are kept where x^2 and e^2 stay in its
    range; the parameter path alone is also exercised with denormal and huge ranges."""
    n = TILE + 9
    check_specs(ctx, [Spec(randn(n, 41) * 1e-12, 1, 1, n), Spec(randn(n, 42) * 1e12, 1, 1, n, asym=True),
                      Spec(randn(n, 44).abs() * 1e10, 1, 1, n, asym=True, percentile=0.999)])
    # ranges / parameters / histogram stay bit-exact far outside that range
    xs = [randn(n, 45) * 1e-42, randn(n, 46) * 1e30]
    dev = [x.cuda() for x in xs]
    descs = q.desc_array([q.make_desc(d, None, 1, 1, n, q.PER_TENSOR, q.ASYM_U8, q.PERCENTILE, 0.999)
                          for d in dev])
    cal = ctx.calibrate(descs)
    torch.cuda.synchronize()
    for t, x in enumerate(xs):
        ref = oracle.calibrate_tensor(x.numpy(), 1, 1, n, False, True, 0.999)
        gmin, gmax, gabs, bad, hist, clip, step, inv, off = ref[:9]
        got = lambda a: a[t:t + 1].cpu().numpy().view(np.uint32)[0]
        for a, r in ((cal.gmin, gmin), (cal.gmax, gmax), (cal.step, step), (cal.inv, inv), (cal.offset, off)):
            assert got(a) == r.view(np.uint32)[0]
        assert got(cal.clip) == np.float32(clip).view(np.uint32)
        assert np.array_equal(cal.hist.cpu().numpy().view(np.uint64).reshape(-1, 2048)[t], hist)


# ----------------------------------------------------------------------------------------- rank
def test_rank_is_bit_exact_on_oracle_metrics(ctx):
    rng = np.random.default_rng(5)
    for trial in range(44):
        n = int(rng.integers(1, 120)) if trial < 40 else (512, 513, 1024, 1500)[trial - 40]   # around the staging limit
        sw = rng.uniform(-5, 60, n).round(1); sa = rng.uniform(-5, 60, n).round(1)
        mw = rng.choice([0.0, 1e-6, 1e-5, 3e-4, 2e-3], n); ma = rng.choice([1e-3, 2e-3, 9e-2, 0.5], n)
        if trial % 5 == 0:
            sw[rng.integers(0, n)] = math.inf
        macs = rng.integers(0, 10 ** 9, n).astype(np.uint64)
        pos = np.cumsum(rng.integers(1, 4, n)).astype(np.float64) if trial % 3 == 0 else None
        mode = trial % 2
        rate = int(rng.integers(0, 10001)); kc = int(rng.integers(0, n + 2))
        ro, rk, rn = oracle.rank_layers(sw, mw, sa, ma, macs=macs, pos=pos, select_mode=mode,
                                        keep_count=kc, rate_permyriad=rate)
        dv = lambda a: torch.from_numpy(np.asarray(a)).cuda()
        cfg = q.default_rank_cfg(select_mode=mode, keep_count=kc, rate_permyriad=rate)
        o, k, nk = ctx.rank_layers(dv(sw), dv(mw), dv(sa), dv(ma), dv(macs.view(np.int64)),
                                   None if pos is None else dv(pos), cfg)
        torch.cuda.synchronize()
        assert o.cpu().numpy().view(np.uint32).tolist() == ro.tolist()
        assert k.cpu().numpy().tolist() == rk.tolist() and int(nk) == rn


def test_rank_without_macs_counts_layers(ctx):
    sw = torch.tensor([30.0, 20.0, 25.0, 40.0], dtype=torch.float64).cuda()
    ones = torch.ones(4, dtype=torch.float64).cuda()
    cfg = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=5000)
    o, k, nk = ctx.rank_layers(sw, ones, sw, ones, None, None, cfg)
    ro, rk, rn = oracle.rank_layers(sw.cpu().numpy(), np.ones(4), sw.cpu().numpy(), np.ones(4),
                                    select_mode=1, rate_permyriad=5000)
    assert o.cpu().numpy().view(np.uint32).tolist() == ro.tolist() and int(nk) == rn == 2


# --------------------------------------------------------------------------------- error paths
def test_argument_errors_are_reported_before_launch(ctx):
    x = torch.zeros(64, device="cuda")
    good = q.make_desc(x, None, 1, 1, 64, q.PER_TENSOR, q.SYM_I8)
    bad_enum = q.make_desc(x, None, 1, 1, 64, 7, q.SYM_I8)
    with pytest.raises(q.binding.Qv2Error) as e:
        ctx.calibrate(q.desc_array([good, bad_enum]))
    assert e.value.status == -1
    null_x = q.make_desc(None, None, 1, 1, 64, q.PER_TENSOR, q.SYM_I8)
    with pytest.raises(q.binding.Qv2Error) as e:
        ctx.calibrate(q.desc_array([null_x]))
    assert e.value.status == -2
    mis = q.make_desc(x, None, 1, 1, 32, q.PER_TENSOR, q.SYM_I8); mis.x = x.data_ptr() + 2
    with pytest.raises(q.binding.Qv2Error) as e:
        ctx.calibrate(q.desc_array([mis]))
    assert e.value.status == -3
    badp = q.make_desc(x, None, 1, 1, 64, q.PER_TENSOR, q.ASYM_U8, q.PERCENTILE, 1.5)
    with pytest.raises(q.binding.Qv2Error) as e:
        ctx.calibrate(q.desc_array([badp]))
    assert e.value.status == -1
    raw_no_y = q.make_desc(x, None, 1, 1, 64, q.PER_TENSOR, q.ASYM_U8, flags=q.PAIR_RAW)
    with pytest.raises(q.binding.Qv2Error):
        ctx.calibrate(q.desc_array([raw_no_y]))
    z = torch.zeros(8193, dtype=torch.float64, device="cuda")     # more layers than supported
    with pytest.raises(q.binding.Qv2Error) as e:
        ctx.rank_layers(z, z, z, z)
    assert e.value.status == -4
    # the context is still usable afterwards
    check_specs(ctx, [Spec(randn(500, 3), 1, 1, 500)])


def test_rank_at_the_maximum_layer_count(ctx):
    rng = np.random.default_rng(11)
    n = 8192
    sw = rng.uniform(10, 60, n).round(2); sa = rng.uniform(10, 60, n).round(2)
    mw = rng.uniform(1e-6, 1e-4, n); ma = rng.uniform(1e-4, 1e-2, n)
    ma[[5, 4000, 8191]] = [3.0, 5.0, 4.0]                       # three MSE outliers
    macs = rng.integers(1, 2 ** 40, n).astype(np.uint64)
    ro, rk, rn = oracle.rank_layers(sw, mw, sa, ma, macs=macs, select_mode=1, rate_permyriad=7000)
    dv = lambda a: torch.from_numpy(np.asarray(a)).cuda()
    cfg = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=7000)
    o, k, nk = ctx.rank_layers(dv(sw), dv(mw), dv(sa), dv(ma), dv(macs.view(np.int64)), None, cfg)
    torch.cuda.synchronize()
    assert o.cpu().numpy().view(np.uint32).tolist() == ro.tolist()
    assert ro.tolist()[:3] == [4000, 8191, 5]
    assert k.cpu().numpy().tolist() == rk.tolist() and int(nk) == rn


def test_tensor_with_more_than_2_to_32_elements(ctx):
    """64-bit element indexing: a 17 GB tensor whose extremes sit beyond element 2^32, checked by
    invariants (the oracle would need minutes): planted min/max, histogram total, and the sum of
    squared errors of the whole against those of its two halves under the same parameters."""
    n = (1 << 32) + 3 * TILE + 5
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * 2 ** 30:
        pytest.skip("needs about 40 GiB of free device memory")
    g = torch.Generator(device="cuda"); g.manual_seed(17)
    x = torch.empty(n, dtype=torch.float32, device="cuda")
    step_n = 1 << 28
    for s in range(0, n, step_n):
        e = min(n, s + step_n)
        x[s:e].normal_(generator=g)
    x[(1 << 32) + 7] = -9.5
    x[n - 1] = 11.25
    d_whole = q.make_desc(x, None, 1, 1, n, q.PER_TENSOR, q.ASYM_U8, q.PERCENTILE, 0.9999)
    cal = ctx.calibrate(q.desc_array([d_whole]))
    torch.cuda.synchronize()
    assert float(cal.gmin[0]) == -9.5 and float(cal.gmax[0]) == 11.25 and int(cal.nonfinite[0]) == 0
    hist = cal.hist.cpu().numpy().view(np.uint64)[:2048]
    assert int(hist.sum()) == n and hist[2047] >= 1
    h1 = 1 << 31
    halves = [q.make_desc(x, None, 1, 1, n, q.PER_TENSOR, q.ASYM_U8, q.MINMAX),
              q.make_desc(x[:h1], None, 1, 1, h1, q.PER_TENSOR, q.ASYM_U8, q.MINMAX),
              q.make_desc(x[h1:], None, 1, 1, n - h1, q.PER_TENSOR, q.ASYM_U8, q.MINMAX)]
    rep = lambda t: t[:1].repeat(3)
    met = ctx.quant_metrics(q.desc_array(halves), rep(cal.step), rep(cal.inv), rep(cal.offset))
    torch.cuda.synchronize()
    sse, sig = met.sse.tolist(), met.sig.tolist()
    assert abs(sse[0] - (sse[1] + sse[2])) <= 1e-7 * sse[0]
    assert abs(sig[0] - (sig[1] + sig[2])) <= 1e-7 * sig[0]
    assert abs(sig[0] / n - 1.0) < 1e-3                         # unit-variance data
    assert abs(float(met.mse[0]) - sse[0] / n) <= 1e-15 * sse[0]
    del x
    torch.cuda.empty_cache()


# --------------------------------------------------------------------------------------- cosine
def test_cosine_similarity_matches_oracle(ctx):
    """Eq. 8 through qv2_quant_metrics_ex.  The three sums behind it (sig, sse, sum x*e) each carry
    the relative error of a 16-term binary32 chain (~1e-7 at worst), so cos agrees to 1e-7
    absolute whatever the operands; for quantization error proper cos sits within ~1e-5 of 1 and
    the sums that matter are tiny against sig, so 1 - cos is compared too, to 1e-4 relative."""
    from parity import make_descs, to_dev
    n = 6 * TILE + 77
    x = randn(n, 61); y = x + 0.05 * randn(n, 62)
    xr = x.clamp_min(0)
    w = randn(70 * 1153, 63) * torch.exp(randn(70, 64)).repeat_interleave(1153)
    specs = [Spec(x, 1, 1, n), Spec(x, 1, 1, n, asym=True), Spec(xr, 1, 1, n, asym=True, percentile=0.999),
             Spec(x, 1, 1, n, asym=True, y=y), Spec(x, 1, 1, n, asym=True, y=y, raw=True),
             Spec(x, 1, 1, n, asym=True, y=-y, raw=True),
             Spec(w, 1, 70, 1153, per_channel=True), Spec(torch.zeros(100), 1, 1, 100)]
    dx = [to_dev(s.x) for s in specs]; dy = [to_dev(s.y) for s in specs]
    descs = make_descs(specs, dx, dy, store_codes=False)
    cal = ctx.calibrate(descs)
    plain = ctx.quant_metrics(descs, cal.step, cal.inv, cal.offset)
    met = ctx.quant_metrics(descs, cal.step, cal.inv, cal.offset, want_cosine=True)
    torch.cuda.synchronize()
    for k in ("sse", "sig", "mse", "sqnr_db"):        # the extra accumulator changes nothing else
        assert torch.equal(getattr(plain, k).view(torch.int64), getattr(met, k).view(torch.int64)), k
    g = 0
    for t, s in enumerate(specs):
        ng = s.channels if s.per_channel else 1
        sl = slice(g, g + ng); g += ng
        mode = oracle.PAIR_SELF if s.y is None else (oracle.PAIR_RAW if s.raw else oracle.PAIR_REQUANT)
        ref = oracle.cosine(s.x.numpy(), None if s.y is None else s.y.numpy(), s.outer, s.channels, s.inner,
                            s.per_channel, s.asym, mode, cal.step[sl].cpu().numpy(), cal.inv[sl].cpu().numpy(),
                            cal.offset[sl].cpu().numpy())
        got = float(met.cosine[t])
        assert abs(got - ref) <= 1e-7, (t, got, ref)
        if 1e-9 < abs(1 - ref) < 1e-2:
            assert abs((1 - got) - (1 - ref)) <= 1e-4 * abs(1 - ref), (t, 1 - got, 1 - ref)
    assert float(met.cosine[5]) < -0.99 and float(met.cosine[7]) == 0.0
    assert 0.9999 < float(met.cosine[0]) < 1.0


# ------------------------------------------------------------------------ fusion-aware ranking
def test_fused_rank_is_bit_exact_on_oracle_metrics(ctx):
    rng = np.random.default_rng(23)
    NG = oracle.NO_GROUP
    for trial in range(40):
        n = int(rng.integers(1, 150)) if trial < 38 else (1024, 2000)[trial - 38]
        sw = rng.uniform(-5, 60, n).round(1); sa = rng.uniform(-5, 60, n).round(1)
        mw = rng.choice([0.0, 1e-6, 1e-5, 3e-4, 2e-3], n); ma = rng.choice([1e-3, 2e-3, 9e-2, 0.5], n)
        n_groups = max(1, n // 4)
        fg = np.where(rng.random(n) < 0.5, NG, rng.integers(0, n_groups, n)).astype(np.uint32)
        macs = rng.integers(0, 10 ** 9, n).astype(np.uint64)
        mode = trial % 2
        rate = int(rng.integers(0, 10001)); kc = int(rng.integers(0, n + 2))
        ro, rk, rn = oracle.rank_layers_fused(sw, mw, sa, ma, fg, macs=macs, select_mode=mode,
                                              keep_count=kc, rate_permyriad=rate)
        dv = lambda a: torch.from_numpy(np.asarray(a)).cuda()
        cfg = q.default_rank_cfg(select_mode=mode, keep_count=kc, rate_permyriad=rate)
        o, k, nk = ctx.rank_layers(dv(sw), dv(mw), dv(sa), dv(ma), dv(macs.view(np.int64)), None, cfg,
                                   fuse_group=dv(fg.view(np.int32)))
        torch.cuda.synchronize()
        assert o.cpu().numpy().view(np.uint32).tolist() == ro.tolist(), trial
        assert k.cpu().numpy().tolist() == rk.tolist() and int(nk) == rn, trial
    # everyone alone: identical to the plain call
    fg = torch.full((n,), -1, dtype=torch.int32, device="cuda")
    a = ctx.rank_layers(dv(sw), dv(mw), dv(sa), dv(ma), dv(macs.view(np.int64)), None, cfg)
    b = ctx.rank_layers(dv(sw), dv(mw), dv(sa), dv(ma), dv(macs.view(np.int64)), None, cfg, fuse_group=fg)
    torch.cuda.synchronize()
    assert all(torch.equal(u, v) for u, v in zip(a, b))


# ---------------------------------------------------------------------------------- bit widths
@pytest.mark.parametrize("bits", [2, 3, 4, 6, 7, 12, 16])
def test_other_bit_widths(ctx, bits):
    n = 3 * TILE + 123
    x = randn(n, 70 + bits); y = x + 0.02 * randn(n, 90 + bits)
    w = randn(40 * 300, 71 + bits) * torch.exp(randn(40, 72)).repeat_interleave(300)
    check_specs(ctx, [Spec(x, 1, 1, n, bits=bits), Spec(x, 1, 1, n, asym=True, bits=bits),
                      Spec(x.clamp_min(0), 1, 1, n, asym=True, percentile=0.999, bits=bits),
                      Spec(x, 1, 1, n, asym=True, y=y, bits=bits),
                      Spec(w, 1, 40, 300, per_channel=True, bits=bits)])


def test_bit_width_argument_errors(ctx):
    x = torch.zeros(64, device="cuda")
    for bad in (1, 17, 200):
        d = q.make_desc(x, None, 1, 1, 64, q.PER_TENSOR, q.SYM_I8, bits=bad)
        with pytest.raises(q.binding.Qv2Error) as e:
            ctx.calibrate(q.desc_array([d]))
        assert e.value.status == -1
    d = q.make_desc(x, None, 1, 1, 64, q.PER_TENSOR, q.SYM_I8, flags=q.STORE_CODES, bits=12)
    with pytest.raises(q.binding.Qv2Error) as e:
        ctx.calibrate(q.desc_array([d]))
    assert e.value.status == -8


# --------------------------------------------------------------------------- integer zero point
@pytest.mark.parametrize("bits", [8, 4])
def test_integer_zero_point_scheme(ctx, bits):
    n = 4 * TILE + 57
    x = randn(n, 110) * 0.8 + 0.3; y = x + 0.02 * randn(n, 111)
    xr = x.clamp_min(0)
    pos = randn(n, 112).abs() + 2.0
    w = randn(30 * 500, 113) * torch.exp(randn(30, 114)).repeat_interleave(500) + 0.1
    specs = [Spec(x, 1, 1, n, zp=True, asym=True, bits=bits),
             Spec(xr, 1, 1, n, zp=True, asym=True, percentile=0.999, bits=bits),
             Spec(pos, 1, 1, n, zp=True, asym=True, bits=bits),            # range widened down to 0
             Spec(-pos, 1, 1, n, zp=True, asym=True, bits=bits),
             Spec(x, 1, 1, n, zp=True, asym=True, y=y, bits=bits),
             Spec(w, 1, 30, 500, per_channel=True, zp=True, asym=True, bits=bits),
             Spec(torch.zeros(500), 1, 1, 500, zp=True, asym=True, bits=bits)]
    cal, met = check_specs(ctx, specs)
    top = float(2 ** bits - 1)
    z = cal.offset.cpu().numpy()
    assert (z == np.rint(z)).all() and z.min() >= 0 and z.max() <= top     # zero points are integer codes
    assert z[2] == 0.0 and z[3] == top


# ------------------------------------------------------------------------------- KL divergence
def test_kl_divergence_matches_oracle(ctx):
    """Eq. 9 on 128 smoothed bins: the two histograms are integers and must match exactly; the
    divergence itself differs only through log() (1 ulp) and is compared to 1e-12 absolute."""
    from parity import make_descs, to_dev
    n = 5 * TILE + 311
    x = randn(n, 131); y = x + 0.05 * randn(n, 132)
    xr = x.clamp_min(0)
    w = randn(50 * 700, 133) * torch.exp(randn(50, 134)).repeat_interleave(700)
    xn = x.clone(); xn[7] = float("nan"); xn[TILE + 1] = float("inf")
    specs = [Spec(x, 1, 1, n), Spec(x, 1, 1, n, asym=True), Spec(x, 1, 1, n, asym=True, zp=True),
             Spec(xr, 1, 1, n, asym=True, percentile=0.999), Spec(x, 1, 1, n, asym=True, y=y),
             Spec(x, 1, 1, n, asym=True, y=y, raw=True), Spec(x, 1, 1, n, bits=4),
             Spec(w, 1, 50, 700, per_channel=True), Spec(x[: 6 * (n // 6)], 2, 3, n // 6, per_channel=True, asym=True),
             Spec(torch.zeros(300), 1, 1, 300), Spec(xn, 1, 1, n, asym=True, y=y, raw=True)]
    dx = [to_dev(s.x) for s in specs]; dy = [to_dev(s.y) for s in specs]
    descs = make_descs(specs, dx, dy, store_codes=False)
    cal = ctx.calibrate(descs)
    kl, hists = ctx.kl_divergence(descs, cal.step, cal.inv, cal.offset, cal.gabsmax)
    kl2, _ = ctx.kl_divergence(descs, cal.step, cal.inv, cal.offset, cal.gabsmax, want_hists=False)
    torch.cuda.synchronize()
    assert torch.equal(kl.view(torch.int64), kl2.view(torch.int64))
    hists = hists.cpu().numpy().view(np.uint64)
    g = 0
    for t, s in enumerate(specs):
        ng = s.channels if s.per_channel else 1
        sl = slice(g, g + ng); g += ng
        mode = oracle.PAIR_SELF if s.y is None else (oracle.PAIR_RAW if s.raw else oracle.PAIR_REQUANT)
        A = float(cal.gabsmax[sl].max())
        ref, hp, hq = oracle.kl_divergence(s.x.numpy(), None if s.y is None else s.y.numpy(), s.outer,
                                           s.channels, s.inner, s.per_channel, 2 if s.zp else s.asym, mode,
                                           cal.step[sl].cpu().numpy(), cal.inv[sl].cpu().numpy(),
                                           cal.offset[sl].cpu().numpy(), A, bits=s.bits)
        assert np.array_equal(hists[t, 0], hp), (t, "hist of x")
        assert np.array_equal(hists[t, 1], hq), (t, "hist of the compared tensor")
        assert abs(float(kl[t]) - ref) <= 1e-12, (t, float(kl[t]), ref)
    assert float(kl[6]) > 5 * float(kl[0]) > 0                 # 4 bits is further from x than 8 bits
    assert int(hists[10, 0].sum()) == n - 2                    # non-finite elements are skipped


# ----------------------------------------------------------------------------- Conv+BN folding
@pytest.mark.parametrize("c,k,mis", [(64, 576, 0), (37, 1153, 0), (5, 25088, 0), (960, 9, 0), (16, 64, 1)])
def test_fold_batchnorm_is_bit_exact(ctx, c, k, mis):
    from parity import to_dev
    w = randn(c * k, 140 + c).reshape(c, k); b = randn(c, 141)
    gamma = torch.rand(c, generator=_g(142)) * 1.5 + 0.5; beta = randn(c, 143)
    mean = randn(c, 144); var = torch.rand(c, generator=_g(145)) * 3 + 0.05
    ra, rc = oracle.fold_batchnorm(w.numpy(), b.numpy(), gamma.numpy(), beta.numpy(), mean.numpy(), var.numpy())
    dw = to_dev(w, mis).view(c, k)
    a, cc = ctx.fold_batchnorm(dw, b.cuda(), gamma.cuda(), beta.cuda(), mean.cuda(), var.cuda())
    a0, c0 = ctx.fold_batchnorm(dw, None, gamma.cuda(), beta.cuda(), mean.cuda(), var.cuda())
    torch.cuda.synchronize()
    assert np.array_equal(a.cpu().numpy().view(np.uint32), ra.view(np.uint32))
    assert np.array_equal(cc.cpu().numpy().view(np.uint32), rc.view(np.uint32))
    r0 = oracle.fold_batchnorm(w.numpy(), None, gamma.numpy(), beta.numpy(), mean.numpy(), var.numpy())[1]
    assert torch.equal(a0, a) and np.array_equal(c0.cpu().numpy().view(np.uint32), r0.view(np.uint32))
    # the folded weights feed the sweep like any other weight tensor
    check_specs(ctx, [Spec(a.cpu(), 1, c, k, per_channel=True)], twice=False)


# ----------------------------------------------------------------------------- 16-bit input types
@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
@pytest.mark.parametrize("mis", [0, 1, 3])
def test_half_precision_inputs(ctx, dtype, mis):
    """binary16 / bfloat16 tensors: values are widened exactly, everything else is the binary32
    definition, so the oracle is fed the stored values and the same bars apply."""
    n = 4 * TILE + 203
    x = randn(n, 150); y = x + 0.03 * randn(n, 151)
    xr = x.clamp_min(0)
    w = randn(48 * 577, 152) * torch.exp(randn(48, 153)).repeat_interleave(577)
    wl = randn(3 * 20001, 154)
    specs = [Spec(x, 1, 1, n, dtype=dtype), Spec(x, 1, 1, n, asym=True, dtype=dtype),
             Spec(xr, 1, 1, n, asym=True, percentile=0.999, dtype=dtype),
             Spec(x, 1, 1, n, asym=True, y=y, dtype=dtype), Spec(x, 1, 1, n, asym=True, y=y, raw=True, dtype=dtype),
             Spec(w, 1, 48, 577, per_channel=True, dtype=dtype), Spec(wl, 1, 3, 20001, per_channel=True, dtype=dtype),
             Spec(x, 1, 1, n, asym=True, zp=True, bits=4, dtype=dtype), Spec(x[:7], 1, 1, 7, dtype=dtype)]
    check_specs(ctx, specs, misalign_x=mis, misalign_y=(mis + 2) % 4 if mis else 0)


def test_half_precision_nonfinite_and_mixed_batch(ctx):
    n = 2 * TILE + 11
    x = randn(n, 160)
    xh = x.clone(); xh[3] = float("inf"); xh[n - 2] = float("nan")
    cal, _ = check_specs(ctx, [Spec(xh, 1, 1, n, asym=True, percentile=0.99, dtype=torch.float16),
                               Spec(x, 1, 1, n, dtype=torch.float32), Spec(x, 1, 1, n, dtype=torch.bfloat16)],
                         check_codes=False)
    assert cal.nonfinite.tolist() == [2, 0, 0]
    big = torch.tensor([70000.0, 1.0]).repeat(50)            # overflows binary16: stored as Inf
    cal, _ = check_specs(ctx, [Spec(big, 1, 1, 100, dtype=torch.float16)], check_codes=False)
    assert int(cal.nonfinite[0]) == 50


# ------------------------------------------------------------ per-channel percentile (own histograms)
def _scaled_channels(o, c, i, seed, relu=False):
    """Channels whose scales differ by orders of magnitude, the case the per-group clip is for."""
    x = torch.randn(o, c, i, generator=_g(seed)) * (10.0 ** torch.linspace(-2, 2, c))[None, :, None]
    return x.clamp_min(0) if relu else x


def test_group_percentile_long_rows_short_rows_and_batches(ctx):
    specs = []
    for (o, c, i), seed in (((1, 3, 3 * TILE + 100), 201),        # rows cut into several one-group tiles
                            ((4, 5, 5000), 202),                  # one tile per row, groups revisited per batch item
                            ((1, 96, 1153), 203),                 # short ragged rows, several per tile
                            ((8, 20, 49), 204),                   # 7x7 maps: 334 rows per tile
                            ((3, 7, 1), 205),                     # one element per row
                            ((2, 2, 4096), 206),                  # exactly at the row-tile threshold
                            ((1, 2, (1 << 22) + 77), 207),        # rows longer than one unit segment
                            ((70, 3, 2047), 208), ((3, 3, 2048), 209)):   # around the warp / CTA segment switch
        for asym, zp, p in ((False, False, 0.999), (True, False, 0.99), (False, True, 0.95)):
            specs.append(Spec(_scaled_channels(o, c, i, seed, relu=asym), o, c, i, per_channel=True, asym=asym, zp=zp,
                              percentile=p, group_pct=True, name=f"group-pct {o}x{c}x{i} asym={asym} zp={zp}"))
    check_specs(ctx, specs)
    check_specs(ctx, specs[:6], misalign_x=3, check_codes=False)


def test_group_percentile_mixed_with_other_modes_keeps_the_layouts_apart(ctx):
    """Per-group histograms exist only for the tensors that ask for them, in descriptor order; the
    per-tensor histograms, the plain modes and the pair mode around them must be untouched."""
    n = 2 * TILE + 33
    a = _scaled_channels(2, 6, 3000, 211, relu=True)
    specs = [Spec(randn(n, 212), 1, 1, n, asym=True, percentile=0.999),
             Spec(a, 2, 6, 3000, per_channel=True, asym=True, percentile=0.99, group_pct=True,
                  y=a + 0.01 * torch.randn(a.shape, generator=_g(213))),
             Spec(randn(64 * 300, 214), 1, 64, 300, per_channel=True),
             Spec(randn(n, 215), 1, 1, n, asym=True, percentile=0.9, group_pct=True),     # per tensor: same as PERCENTILE
             Spec(_scaled_channels(1, 4, 20000, 216), 1, 4, 20000, per_channel=True, percentile=0.9999, group_pct=True),
             Spec(_scaled_channels(2, 6, 3000, 217), 2, 6, 3000, per_channel=True, percentile=0.99)]  # tensor-level clip
    cal, _ = check_specs(ctx, specs)
    assert int(q.lib().qv2_group_hist_count(q.desc_array([]), 0)) == 0


def test_group_percentile_nonfinite_constant_and_empty_groups(ctx):
    o, c, i = 2, 4, 6000
    x = _scaled_channels(o, c, i, 221)
    x[0, 1, 17] = float("nan"); x[1, 1, 5999] = float("inf")     # skipped in channel 1's histogram
    x[:, 2, :] = 0.0                                             # absmax 0: everything in bin 0, degenerate range
    x[:, 3, :] = -3.5                                            # constant: one bin, clip = absmax
    specs = [Spec(x, o, c, i, per_channel=True, percentile=0.99, group_pct=True),
             Spec(x[:, :, :77].contiguous(), o, c, 77, per_channel=True, asym=True, percentile=0.99, group_pct=True),
             Spec(torch.zeros(0), 1, 5, 0, per_channel=True, percentile=0.5, group_pct=True)]   # no elements at all
    check_specs(ctx, specs, check_codes=False)


_GROUP_WALKER_SHAPES = (
    (64, 300, 1), (4, 37, 7), (2, 5000, 1), (128, 20, 16), (1, 9, 2048),      # packed small groups (up to 2048 elements)
    (129, 3, 16), (6, 8, 196), (64, 4, 784), (3, 5, 12544), (2, 3, 50176),    # whole 16-byte groups: one index space
    (128, 6, 49), (50, 3, 255), (2049, 2, 1),                                 # short rows that do not line up
    (9, 3, 257), (5, 3, 1153), (3, 2, 4097))                                  # one row per warp / per CTA


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
def test_group_percentile_every_unit_walker(ctx, dtype):
    """Per-group histograms are counted by different walkers depending on the group size, the row
    length and whether rows start on 16-byte boundaries; every one must give the oracle's counts,
    with the tensor start shifted off the boundary too, and with non-finite elements skipped."""
    specs = [Spec(_scaled_channels(o, c, i, 260 + k, relu=k % 2 == 1), o, c, i, per_channel=True, asym=k % 2 == 1,
                  percentile=0.99, group_pct=True, dtype=dtype, name=f"group-pct {o}x{c}x{i} {dtype}")
             for k, (o, c, i) in enumerate(_GROUP_WALKER_SHAPES)]
    check_specs(ctx, specs, check_codes=False)
    for mis in (1, 2, 3):
        check_specs(ctx, specs, misalign_x=mis, check_codes=False, twice=False)
    bad = []
    for k, s in enumerate(specs):
        x = s.x.clone()
        flat = x.view(-1)
        flat[(7 * k) % flat.numel()] = float("nan")
        flat[flat.numel() - 1 - (3 * k) % flat.numel()] = float("-inf")
        bad.append(Spec(x, s.outer, s.channels, s.inner, per_channel=True, asym=s.asym, percentile=0.99, group_pct=True,
                        dtype=dtype, name=s.name + " nonfinite"))
    check_specs(ctx, bad, check_codes=False, twice=False)


@pytest.mark.parametrize("p", [0.0, 1e-9, 0.1, 0.5, 0.731, 1.0 - 1e-12, 1.0])
def test_group_percentile_any_percentile(ctx, p):
    """The per-group clip is found by a scan from the top bin down; the bin must be the one the
    cumulative-count rule names for percentiles anywhere in [0, 1], with and without skipped
    (non-finite) elements, where the group's count is no longer its size."""
    x = _scaled_channels(3, 9, 2500, 251, relu=True)
    xn = x.clone(); xn[1, 4, 100] = float("nan"); xn[2, 0, 7] = float("-inf")
    specs = [Spec(x, 3, 9, 2500, per_channel=True, asym=True, percentile=p, group_pct=True),
             Spec(xn, 3, 9, 2500, per_channel=True, percentile=p, group_pct=True),
             Spec(randn(5 * 40, 252), 1, 5, 40, per_channel=True, percentile=p, group_pct=True)]
    check_specs(ctx, specs, check_codes=False)


@pytest.mark.parametrize("dtype", [torch.float16, torch.bfloat16])
def test_group_percentile_sixteen_bit_inputs(ctx, dtype):
    specs = [Spec(_scaled_channels(2, 5, 9000, 231), 2, 5, 9000, per_channel=True, percentile=0.999, group_pct=True, dtype=dtype),
             Spec(_scaled_channels(3, 33, 200, 232, relu=True), 3, 33, 200, per_channel=True, asym=True, percentile=0.99,
                  group_pct=True, dtype=dtype)]
    check_specs(ctx, specs, check_codes=False)
    check_specs(ctx, specs, misalign_x=1, check_codes=False)


def test_group_percentile_in_the_chained_pass_and_its_graph(ctx):
    """qv2_sweep_model and the captured pass accept the mode (histograms stay in context scratch)."""
    w = randn(32 * 500, 241)
    a = _scaled_channels(4, 32, 400, 242, relu=True)
    y = a + 0.02 * torch.randn(a.shape, generator=_g(243))
    dw, da, dy = w.cuda(), a.reshape(-1).cuda(), y.reshape(-1).cuda()
    descs = q.desc_array([q.make_desc(dw, None, 1, 32, 500, q.PER_CHANNEL, q.SYM_I8),
                          q.make_desc(da, dy, 4, 32, 400, q.PER_CHANNEL, q.ASYM_U8, q.PERCENTILE_GROUP, 0.99)])
    cfg = q.default_rank_cfg(select_mode=q.BY_COUNT, keep_count=1)
    macs = torch.ones(1, dtype=torch.int64, device="cuda")
    sb, t = ctx.alloc_sweep_buffers(descs, 1)
    ctx.sweep_model(descs, 1, macs, None, cfg, sb)
    torch.cuda.synchronize()
    ref = oracle.sweep_tensor(a.numpy().reshape(-1), y.numpy().reshape(-1), 4, 32, 400, True, True, 0.99,
                              group_percentile=True)
    assert np.array_equal(t["step"][32:64].cpu().numpy().view(np.uint32), ref.step.view(np.uint32))
    assert_metric_close(float(t["mse"][1]), float(t["sqnr_db"][1]), ref.mse, ref.sqnr_db, "chained group-pct")
    first = [float(t["mse"][1]), float(t["sqnr_db"][1])]
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        gctx = q.Context(0, stream=s)
        try:
            sb2, t2 = gctx.alloc_sweep_buffers(descs, 1)
            graph = gctx.sweep_graph(descs, 1, macs, None, cfg, sb2)
            t2["mse"].zero_(); t2["step"].zero_()
            graph.launch()
            s.synchronize()
            assert [float(t2["mse"][1]), float(t2["sqnr_db"][1])] == first
            assert torch.equal(t2["step"], t["step"])
        finally:
            gctx.close()


# ------------------------------------------------- the row walkers and the row lengths at which they change
@pytest.mark.parametrize("inner", [1, 2, 3, 4, 5, 7, 8, 9, 13, 27, 49, 127, 128, 196, 319, 320, 321, 510, 511, 512, 513, 1021])
def test_short_rows_per_channel_all_modes(ctx, inner):
    """The range kernel walks rows below 320 elements lane-contiguously (32 consecutive elements per
    thread) and longer ones in per-warp chunks; the metrics kernel fetches parameters per 16-byte
    group below 512 elements per row (per element below 4) and walks longer rows in per-warp
    chunks.  Lengths on both sides of every switch, multiples of four and not.  Self, re-quantized
    pair and raw pair, symmetric / affine / zero point, with codes, several batch items so that a
    channel's rows are far apart."""
    o, c = 5, 37
    n = o * c * inner
    x = _scaled_channels(o, c, inner, 300 + inner)
    y = x + 0.01 * x.abs().mean() * torch.randn(x.shape, generator=_g(400 + inner))
    specs = [Spec(x, o, c, inner, per_channel=True, name="self sym"),
             Spec(x, o, c, inner, per_channel=True, asym=True, name="self affine"),
             Spec(x, o, c, inner, per_channel=True, zp=True, name="self zero point"),
             Spec(x, o, c, inner, per_channel=True, asym=True, y=y, name="pair requant"),
             Spec(x, o, c, inner, per_channel=True, zp=True, y=y, name="pair requant zero point"),
             Spec(x, o, c, inner, per_channel=True, y=y, raw=True, name="pair raw"),
             Spec(x, o, c, inner, per_channel=True, bits=4, name="4 bit"),
             Spec(x.clamp_min(0), o, c, inner, per_channel=True, asym=True, percentile=0.99, group_pct=True,
                  name="own percentile per channel")]
    check_specs(ctx, specs)
    check_specs(ctx, specs[:6], misalign_x=1, misalign_y=2, check_codes=False)
    half = [Spec(s.x, s.outer, s.channels, s.inner, per_channel=True, asym=s.asym, zp=s.zp, y=s.y, raw=s.raw,
                 dtype=torch.bfloat16, name=s.name + " bf16") for s in specs[:6]]
    check_specs(ctx, half, check_codes=False)


def test_short_rows_with_nonfinite_elements_and_many_rows_per_tile(ctx):
    o, c, inner = 3, 2000, 9                      # 6000 rows: four tiles of 1820 rows
    x = _scaled_channels(o, c, inner, 501)
    x[0, 5, 3] = float("nan"); x[2, 1999, 8] = float("-inf"); x[1, 0, 0] = float("inf")
    x[:, 7, :] = 0.0
    check_specs(ctx, [Spec(x, o, c, inner, per_channel=True), Spec(x, o, c, inner, per_channel=True, asym=True)],
                check_codes=False)
    o, c, inner = 4, 300, 50                      # rows that straddle 16-byte groups, a row without a finite element
    z = _scaled_channels(o, c, inner, 502)
    z[1, 17, :] = float("nan"); z[0, 17, :] = float("inf"); z[2, 17, :] = float("-inf"); z[3, 17, :] = float("nan")
    z[3, 299, 49] = float("inf"); z[0, 0, 0] = float("nan"); z[2, 100, 3:5] = float("nan")
    for mis in (0, 1, 3):
        check_specs(ctx, [Spec(z, o, c, inner, per_channel=True), Spec(z, o, c, inner, per_channel=True, asym=True)],
                    misalign_x=mis, check_codes=False, twice=False)


# ----------------------------------------------------------------------- seeded random descriptor sets
@pytest.mark.parametrize("seed", [1, 2, 3, 4, 5, 6])
def test_random_descriptor_sets_in_one_batched_call(ctx, seed):
    """Forty tensors of random shape, granularity, scheme, range mode, bit width, storage type and
    pair mode in ONE calibrate and ONE metrics call: every combination of row walker (flat, warp
    per row, element per thread) and tile kind meets every arithmetic variant, and the planner has
    to keep their groups, slots and histograms apart."""
    rng = np.random.default_rng(1000 + seed)
    inner_pool = [1, 2, 3, 7, 9, 31, 32, 33, 49, 100, 127, 128, 129, 196, 318, 322, 500, 514, 784, 1153, 3136, 4095, 4096,
                  4097, 12544, 16383, 16384, 16385, 40000]
    specs = []
    total = 0
    while len(specs) < 40 and total < 6_000_000:
        inner = int(rng.choice(inner_pool))
        per_channel = bool(rng.random() < 0.7)
        c = int(rng.integers(1, 40 if inner > 1000 else 300))
        o = int(rng.integers(1, 5))
        if o * c * inner > 1_500_000:
            c = max(1, 1_500_000 // (o * inner))
        n = o * c * inner
        total += n
        scheme = int(rng.integers(0, 3))
        x = _scaled_channels(o, c, inner, int(rng.integers(1 << 30)), relu=bool(rng.random() < 0.4))
        if rng.random() < 0.1:
            x = x * 0.0 + 1.25                        # constant tensor
        pair = rng.random() < 0.5
        y = x + 0.02 * float(x.abs().mean() + 1e-6) * torch.randn(x.shape, generator=_g(int(rng.integers(1 << 30)))) \
            if pair else None
        pct = float(rng.choice([0.9, 0.99, 0.9999, 1.0])) if rng.random() < 0.5 else None
        specs.append(Spec(x, o, c, inner, per_channel=per_channel, asym=scheme == 1, zp=scheme == 2, percentile=pct,
                          group_pct=pct is not None and rng.random() < 0.5, y=y, raw=bool(pair and rng.random() < 0.25),
                          bits=int(rng.choice([8, 8, 8, 4, 2, 12, 16])),
                          dtype=[torch.float32, torch.float32, torch.float16, torch.bfloat16][int(rng.integers(0, 4))],
                          name=f"seed {seed} tensor {len(specs)}: {o}x{c}x{inner} pc={per_channel} scheme={scheme}"))
    order = rng.permutation(len(specs))
    specs = [specs[i] for i in order]
    check_specs(ctx, specs, misalign_x=int(rng.integers(0, 4)), misalign_y=int(rng.integers(0, 4)),
                check_codes=bool(seed % 2))
