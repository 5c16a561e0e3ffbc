"""Pins for the CPU oracle: each function is checked against something other than itself --
closed forms, exact constructions in which every operation is exact, library routines on
special cases, brute force with Python integers / fractions, and invariants.  A dropped term,
a wrong sign or index, or a transposed operand in the oracle fails at least one test here.
No GPU is involved."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(20250107)


# ----------------------------------------------------------------------------------- ranges
def test_ranges_match_numpy_per_tensor_and_per_channel():
    o, c, i = 3, 5, 7
    x = RNG.standard_normal((o, c, i)).astype(np.float32)
    mn, mx, am, bad = oracle.ranges(x, o, c, i, False)
    assert bad == 0 and mn[0] == x.min() and mx[0] == x.max()
    assert am[0] == np.abs(x).max()
    mn, mx, am, bad = oracle.ranges(x, o, c, i, True)
    # channel is the MIDDLE axis: a transposed view must not match unless indexing is right
    np.testing.assert_array_equal(mn, x.min(axis=(0, 2)))
    np.testing.assert_array_equal(mx, x.max(axis=(0, 2)))
    np.testing.assert_array_equal(am, np.abs(x).max(axis=(0, 2)))
    assert not np.array_equal(mn, x.reshape(o, i, c).min(axis=(0, 1)))


def test_ranges_planted_extremes_first_last_and_group_boundary():
    c, i = 4, 9
    x = np.zeros((1, c, i), np.float32)
    x[0, 0, 0] = -3.0       # first element of the tensor
    x[0, 3, 8] = 5.0        # last element
    x[0, 1, 8] = 7.0        # last element of group 1
    x[0, 2, 0] = -9.0       # first element of group 2
    mn, mx, am, _ = oracle.ranges(x, 1, c, i, True)
    np.testing.assert_array_equal(mn, np.float32([-3, 0, -9, 0]))
    np.testing.assert_array_equal(mx, np.float32([0, 7, 0, 5]))
    np.testing.assert_array_equal(am, np.float32([3, 7, 9, 5]))
    mn, mx, am, _ = oracle.ranges(x, 1, c, i, False)
    assert (mn[0], mx[0], am[0]) == (-9.0, 7.0, 9.0)


def test_ranges_negative_zero_and_nonfinite():
    x = np.float32([-0.0, -0.0, np.nan, np.inf, -np.inf, -0.0])
    mn, mx, am, bad = oracle.ranges(x, 1, 1, 6, False)
    assert bad == 3
    for v in (mn[0], mx[0], am[0]):
        assert v == 0.0 and not np.signbit(v)
    x = np.float32([np.nan, 2.0, -1.0, np.inf])
    mn, mx, am, bad = oracle.ranges(x, 1, 1, 4, False)
    assert (mn[0], mx[0], am[0], bad) == (-1.0, 2.0, 2.0, 2)
    x = np.float32([np.nan, np.nan])
    mn, mx, am, bad = oracle.ranges(x, 1, 2, 1, True)
    assert bad == 2 and not mn.any() and not mx.any() and not am.any()


# -------------------------------------------------------------------------------- histogram
def test_histogram_planted_bin_centres_and_top_edge():
    A = 4.0  # power of two: 2048/A and every product below are exact
    j = np.arange(2048)
    x = ((j + 0.5) * (A / 2048)).astype(np.float32)
    x = np.concatenate([x, -x, np.float32([A, -A])])   # |x| is what is binned
    h = oracle.histogram(x, A)
    expect = np.full(2048, 2, np.uint64)
    expect[2047] += 2                                  # x = +-A lands in the last bin
    np.testing.assert_array_equal(h, expect)
    assert h.sum() == x.size


def test_histogram_ramp_is_flat_and_percentile_closed_form():
    A, per = 8.0, 16
    n = 2048 * per
    x = ((np.arange(n) + 0.5) * (A / n)).astype(np.float32)   # exact: A/n is a power of two
    x[-1] = A                                                 # make A the absmax
    h = oracle.histogram(x, A)
    np.testing.assert_array_equal(h, np.full(2048, per, np.uint64))
    # cumulative count reaches ceil(0.99 n) first in bin k* with (k*+1) >= 0.99*2048 = 2027.52
    clip = oracle.percentile_clip(h, 0.99, A)
    assert clip == np.float32(2028 * A / 2048)
    assert oracle.percentile_clip(h, 1.0, A) == np.float32(A)       # k* = 2047 -> A itself
    assert oracle.percentile_clip(h, 0.0, A) == np.float32(A / 2048)  # T clamps to 1 -> bin 0
    assert oracle.percentile_clip(h, 0.5, A) == np.float32(A / 2)


def test_histogram_zeros_nonfinite_and_degenerate():
    x = np.zeros(1000, np.float32)
    h = oracle.histogram(x, 0.0)
    assert h[0] == 1000 and h[1:].sum() == 0
    assert oracle.percentile_clip(h, 0.9999, 0.0) == 0.0
    # half zeros (post-ReLU): the zero mass sits in bin 0 and pushes the median bin to 0
    x = np.concatenate([np.zeros(500, np.float32), np.linspace(0.5, 1.0, 500, dtype=np.float32)])
    h = oracle.histogram(x, 1.0)
    assert h[0] == 500 and h.sum() == 1000 and h[1:1024].sum() == 0
    assert oracle.percentile_clip(h, 0.5, 1.0) == np.float32(1.0 / 2048)
    x = np.float32([np.nan, np.inf, 0.25, -np.inf, 1.0])
    h = oracle.histogram(x, 1.0)
    assert h.sum() == 2 and h[512] == 1 and h[2047] == 1


def test_histogram_matches_numpy_on_random_data():
    x = (RNG.standard_normal(50_000) * 0.7).astype(np.float32)
    A = np.float32(np.abs(x).max())
    h = oracle.histogram(x, float(A))
    w = np.float32(2048) / A
    b = np.minimum((np.abs(x) * w).astype(np.float32).astype(np.int64), 2047)
    np.testing.assert_array_equal(h, np.bincount(b, minlength=2048).astype(np.uint64))
    # percentile against a direct sort: the clip is the upper edge of the bin holding the
    # T-th smallest |x|
    p = 0.999
    T = math.ceil(p * x.size)
    kth = np.sort(np.abs(x))[T - 1]
    kbin = min(int(np.float32(kth * w)), 2047)
    clip = oracle.percentile_clip(h, p, float(A))
    assert clip == np.float32(np.float32(kbin + 1) * np.float32(A / np.float32(2048)))


# --------------------------------------------------------------------------------- qparams
def test_qparams_symmetric_and_asymmetric_definitions():
    gmin = np.float32([-1.27, 0.0, -2.0]); gmax = np.float32([0.5, 2.55, 6.0])
    gabs = np.maximum(np.abs(gmin), np.abs(gmax))
    step, inv, off = oracle.qparams(False, gmin, gmax, gabs)
    np.testing.assert_array_equal(step, gabs / np.float32(127))
    np.testing.assert_array_equal(inv, np.float32(127) / gabs)
    assert not off.any()
    step, inv, off = oracle.qparams(True, gmin, gmax, gabs)
    d = gmax - gmin
    np.testing.assert_array_equal(step, d / np.float32(255))
    np.testing.assert_array_equal(inv, np.float32(255) / d)
    np.testing.assert_array_equal(off, gmin)
    # percentile clip narrows both schemes
    step, inv, off = oracle.qparams(False, gmin, gmax, gabs, clip=1.0)
    np.testing.assert_array_equal(step, np.minimum(gabs, 1) / np.float32(127))
    step, inv, off = oracle.qparams(True, gmin, gmax, gabs, clip=1.0)
    np.testing.assert_array_equal(off, np.maximum(gmin, -1))
    np.testing.assert_array_equal(step, (np.minimum(gmax, 1) - np.maximum(gmin, -1)) / np.float32(255))
    # degenerate ranges fall back to a unit grid
    z = np.zeros(1, np.float32)
    for asym in (False, True):
        step, inv, off = oracle.qparams(asym, z, z, z)
        assert step[0] == 1.0 and inv[0] == 1.0 and off[0] == 0.0


# ------------------------------------------------------------------------ codes and metrics
def _self(x, per_channel=False, asym=False, shape=None, percentile=None, codes=True):
    x = np.asarray(x, np.float32)
    o, c, i = shape if shape else (1, 1, x.size)
    return oracle.sweep_tensor(x, None, o, c, i, per_channel, asym, percentile, want_codes=codes)


def test_on_grid_tensor_has_zero_error_symmetric():
    d = 2.0 ** -7
    k = np.arange(-127, 128)
    r = _self(k * d)
    np.testing.assert_array_equal(r.codes, k.astype(np.int8))
    assert r.step[0] == np.float32(d) and r.sse == 0.0 and r.mse == 0.0 and r.sqnr_db == math.inf


def test_on_grid_tensor_has_zero_error_asymmetric_with_offset():
    d = 2.0 ** -6
    k = np.arange(0, 256)
    lo = -1.0                      # offset is the real-valued minimum, range need not hold 0
    r = _self(k * d + lo, asym=True)
    np.testing.assert_array_equal(r.codes, k.astype(np.uint8))
    assert r.offset[0] == np.float32(lo) and r.step[0] == np.float32(d)
    assert r.sse == 0.0 and r.sqnr_db == math.inf


def test_exact_ties_round_to_even():
    d = 2.0 ** -7
    k = np.arange(-126, 126)
    x = np.concatenate([(k + 0.5) * d, [127 * d, -127 * d]])     # absmax fixes the grid
    r = _self(x)
    even = np.where(k % 2 == 0, k, k + 1)
    np.testing.assert_array_equal(r.codes[:-2], even.astype(np.int8))
    # every error is exactly half a step
    assert r.sse == pytest.approx(k.size * (d / 2) ** 2, rel=1e-15)


def test_saturation_beyond_percentile_clip():
    # 9999 small values and one huge one: the 99 % clip lands far below the outlier, which
    # must saturate at +127 (symmetric) / 255 (asymmetric) instead of wrapping
    x = np.concatenate([np.linspace(-1, 1, 9999), [50.0, -60.0]]).astype(np.float32)
    r = _self(x, percentile=0.99)
    assert r.clip < 2.0 and r.codes[-2] == 127 and r.codes[-1] == -127
    assert abs(r.codes[:-2].astype(int)).max() <= 127
    r = _self(x, asym=True, percentile=0.99)
    assert r.codes[-2] == 255 and r.codes[-1] == 0


def test_power_of_two_scaling_invariance():
    x = (RNG.standard_normal(20_000)).astype(np.float32)
    for asym in (False, True):
        base = _self(x, asym=asym)
        for m in (-9, 5):
            s = _self(x * np.float32(2.0 ** m), asym=asym)
            np.testing.assert_array_equal(base.codes, s.codes)
            assert s.mse == pytest.approx(base.mse * 4.0 ** m, rel=1e-14)
            assert s.sqnr_db == pytest.approx(base.sqnr_db, abs=1e-10)


def test_codes_agree_with_semantic_double_quantizer():
    """rne(x / Delta) in pure double differs from the binary32 definition only where x/Delta
    sits within rounding error of a tie."""
    x = RNG.standard_normal(400_000).astype(np.float32)
    r = _self(x)
    t = x.astype(np.float64) / (float(r.gabsmax[0]) / 127.0)
    q = np.clip(np.rint(t), -127, 127).astype(np.int64)
    diff = q != r.codes.astype(np.int64)
    assert diff.mean() < 1e-4
    frac = np.abs(t - np.floor(t) - 0.5)
    assert (frac[diff] < 1e-4).all()
    assert np.abs(q - r.codes.astype(np.int64)).max() <= 1


def test_mse_brute_force_python_fractions():
    """Tiny tensor, every step redone with exact rational arithmetic."""
    x = np.float32([0.11, -0.52, 0.9, 0.333, -1.0, 0.75, 0.0, 0.49])
    r = _self(x)
    step = Fraction(float(r.step[0]))
    sse = Fraction(0); sig = Fraction(0)
    for v, q in zip(x, r.codes):
        e = Fraction(float(v)) - int(q) * step
        sse += e * e
        sig += Fraction(float(v)) ** 2
    assert r.sse == pytest.approx(float(sse), rel=1e-15)
    assert r.sig == pytest.approx(float(sig), rel=1e-15)
    assert r.mse == pytest.approx(float(sse / 8), rel=1e-15)
    assert r.sqnr_db == pytest.approx(10 * math.log10(float(sig / sse)), abs=1e-12)
    # the codes themselves: nearest grid point, checked without the oracle's own formula
    for v, q in zip(x, r.codes):
        assert abs(Fraction(float(v)) - int(q) * step) <= step / 2 + Fraction(1, 10 ** 9)


def test_uniform_noise_midpoint_construction_gives_delta_sq_over_12():
    """M equispaced points in every full cell of the symmetric grid: the mean squared error of
    a cell is (Delta^2/12)(1 - 1/M^2) exactly; all values and products are exact in binary32."""
    d, M = 2.0 ** -7, 64
    k = np.arange(-126, 127)[:, None]
    j = np.arange(M)[None, :]
    x = ((k - 0.5) + (j + 0.5) / M) * d
    x = np.concatenate([x.reshape(-1), [127 * d, -127 * d]])
    r = _self(x, codes=False)
    n_cell = 253 * M
    expect = (d * d / 12) * (1 - 1 / M ** 2) * n_cell / (n_cell + 2)
    assert r.mse == pytest.approx(expect, rel=1e-13)


def test_uniform_random_mse_and_sqnr_closed_forms():
    n = 1 << 22
    u = RNG.random(n)
    xs = ((2 * u - 1) * 3.0).astype(np.float32)
    r = _self(xs, codes=False)
    d = float(r.step[0])
    assert r.mse == pytest.approx(d * d / 12, rel=3e-3)
    assert r.sqnr_db == pytest.approx(20 * math.log10(254), abs=0.02)       # 48.097 dB
    xa = (u * 5.0).astype(np.float32)
    r = _self(xa, asym=True, codes=False)
    assert r.sqnr_db == pytest.approx(10 * math.log10(4 * 255 ** 2), abs=0.02)  # 54.151 dB
    assert r.sqnr_db == pytest.approx(10 * math.log10(r.sig / (n * r.mse)), abs=1e-9)


def test_per_channel_uses_the_middle_axis_and_own_scale():
    o, c, i = 2, 3, 5
    x = RNG.standard_normal((o, c, i)).astype(np.float32)
    x[:, 1, :] *= 100.0          # one loud channel
    r = _self(x, per_channel=True, shape=(o, c, i))
    sse = 0.0
    for ch in range(c):
        sub = np.ascontiguousarray(x[:, ch, :])
        rc = _self(sub)
        # codes of channel ch equal a stand-alone per-tensor quantization of that channel
        np.testing.assert_array_equal(r.codes.reshape(o, c, i)[:, ch, :].reshape(-1), rc.codes)
        sse += rc.sse
    assert r.sse == pytest.approx(sse, rel=1e-14)
    rt = _self(x)                # per-tensor: the loud channel sets everyone's step
    assert rt.mse > 2 * r.mse


def test_pair_modes():
    x = RNG.standard_normal(5000).astype(np.float32)
    y = (x + 0.01 * RNG.standard_normal(5000)).astype(np.float32)
    raw = oracle.sweep_tensor(x, y, 1, 1, 5000, False, True, pair_mode=oracle.PAIR_RAW)
    d = x.astype(np.float64) - y.astype(np.float64)
    assert raw.sse == pytest.approx(float((d * d).sum()), rel=1e-14)
    assert raw.sig == pytest.approx(float((x.astype(np.float64) ** 2).sum()), rel=1e-14)
    rq = oracle.sweep_tensor(x, y, 1, 1, 5000, False, True, want_codes=True)
    # parameters come from x; codes are those of y on x's grid; error is x minus dequantized y
    own = oracle.quant_metrics(y, None, 1, 1, 5000, False, True, oracle.PAIR_SELF,
                               rq.step, rq.inv, rq.offset, want_codes=True)
    np.testing.assert_array_equal(rq.codes, own["codes"])
    yhat = rq.codes.astype(np.float64) * float(rq.step[0]) + float(rq.offset[0])
    e = x.astype(np.float64) - yhat
    assert rq.sse == pytest.approx(float((e * e).sum()), rel=1e-14)
    # swapping the operands changes the signal term: SIG is always the reference tensor
    sw = oracle.sweep_tensor(y, x, 1, 1, 5000, False, True, pair_mode=oracle.PAIR_RAW)
    assert sw.sse == pytest.approx(raw.sse, rel=1e-14) and sw.sig != raw.sig
    # y identical to an on-grid x: zero noise
    z = oracle.sweep_tensor(x, x, 1, 1, 5000, False, True, pair_mode=oracle.PAIR_RAW)
    assert z.sse == 0.0 and z.sqnr_db == math.inf
    zero_sig = oracle.sweep_tensor(np.zeros(4, np.float32), np.ones(4, np.float32), 1, 1, 4,
                                   False, True, pair_mode=oracle.PAIR_RAW)
    assert zero_sig.sqnr_db == -math.inf and zero_sig.mse == 1.0


# ------------------------------------------------------------------------------------- rank
def _py_rank(sw, mw, sa, ma, pos=None, wg=2.0, ag=1.0, fac=5.0, cap=200.0):
    """Independent restatement with Python floats and the library sort."""
    n = len(sw)
    cl = lambda v: max(-cap, min(cap, v))
    score, sev = [], []
    mean_w = sum(mw) / n; mean_a = sum(ma) / n
    for i in range(n):
        if i == 0:
            dw = da = 0.0
        else:
            den = (pos[i] - pos[i - 1]) if pos is not None else 1.0
            dw = (cl(sw[i]) - cl(sw[i - 1])) / den
            da = (cl(sa[i]) - cl(sa[i - 1])) / den
        score.append(wg * dw + ag * da)
        rw = mw[i] / mean_w if mean_w > 0 else 0.0
        ra = ma[i] / mean_a if mean_a > 0 else 0.0
        sev.append(max(rw, ra))
    out = sorted([i for i in range(n) if sev[i] > fac], key=lambda i: (-sev[i], i))
    rest = sorted([i for i in range(n) if sev[i] <= fac], key=lambda i: (score[i], i))
    return out + rest


def test_rank_hand_worked_six_layers():
    # SQNR (dB) per layer; deltas: w = [0,-5,+2,-1,+6,-8], a = [0,+1,-4,+3,-2,+1]
    sw = [40.0, 35.0, 37.0, 36.0, 42.0, 34.0]
    sa = [30.0, 31.0, 27.0, 30.0, 28.0, 29.0]
    # score = 2*dw + da = [0,-9,0,1,10,-15]
    mw = [1.0, 1.0, 1.0, 1.0, 1.0, 1.0]
    ma = [1.0, 1.0, 1.0, 1.0, 1.0, 1.0]
    order, keep, nk = oracle.rank_layers(sw, mw, sa, ma, keep_count=2)
    assert order.tolist() == [5, 1, 0, 2, 3, 4]        # tie between layers 0 and 2 keeps layer order
    assert keep.tolist() == [0, 1, 0, 0, 0, 1] and nk == 2
    # layer 3 becomes an MSE outlier (its MSE is > 5x the mean): it jumps to the top
    ma2 = [1.0, 1.0, 1.0, 60.0, 1.0, 1.0]              # mean 10.83, ratio 5.54
    order, _, _ = oracle.rank_layers(sw, mw, sa, ma2)
    assert order.tolist() == [3, 5, 1, 0, 2, 4]
    ma3 = [1.0, 1.0, 1.0, 25.0, 1.0, 1.0]              # mean 5, ratio exactly 5: not an outlier
    order, _, _ = oracle.rank_layers(sw, mw, sa, ma3)
    assert order.tolist() == [5, 1, 0, 2, 3, 4]
    # two outliers: the more severe one first, whichever list it came from
    mw4 = [1.0, 1.0, 100.0, 1.0, 1.0, 1.0]             # ratio 100/17.5 = 5.71
    order, _, _ = oracle.rank_layers(sw, mw4, sa, ma2)
    assert order.tolist()[:2] == [2, 3]


def test_rank_literal_outlier_order_of_algorithm_2():
    """Algorithm 2, RankLayersBySensitivity, as printed: the layer loop inserts every layer whose
    MSE exceeds 5x the mean at the HEAD of the list when it meets it, so among the outliers the
    one met last stands first (reverse layer order), whatever their severities."""
    sw = [40.0, 35.0, 37.0, 36.0, 42.0, 34.0, 33.0, 39.0]
    sa = [30.0, 31.0, 27.0, 30.0, 28.0, 29.0, 30.0, 31.0]
    # three large weight MSEs among eight layers, none above 5x the mean
    mw = [1.0, 80.0, 1.0, 1.0, 100.0, 1.0, 90.0, 1.0]    # mean 34.375; ratios 2.33, 2.91, 2.62: none > 5
    ma = [1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0, 1.0]
    o_sev, _, _ = oracle.rank_layers(sw, mw, sa, ma)
    o_lit, _, _ = oracle.rank_layers(sw, mw, sa, ma, outlier_order=1)
    assert o_sev.tolist() == o_lit.tolist()              # no outlier: the two readings coincide
    # 20 layers so that three large MSEs exceed 5x the mean: mean = (17 + 300 + 500 + 400)/20 = 60.85
    n = 20
    sw = [40.0 - 0.5 * i for i in range(n)]              # all deltas equal: the rest keeps layer order
    sa = [30.0] * n
    mw = [1.0] * n
    mw[3], mw[9], mw[14] = 400.0, 500.0, 310.0           # ratios 6.57, 8.22, 5.09
    ma = [1.0] * n
    o_sev, _, _ = oracle.rank_layers(sw, mw, sa, ma)
    o_lit, k_lit, nk = oracle.rank_layers(sw, mw, sa, ma, outlier_order=1, keep_count=2)
    rest = [i for i in range(n) if i not in (3, 9, 14)]
    # layer 0 has delta 0, the others -0.5*2 = -1: they precede it
    rest_sorted = [i for i in rest if i != 0] + [0]
    assert o_sev.tolist() == [9, 3, 14] + rest_sorted    # by severity
    assert o_lit.tolist() == [14, 9, 3] + rest_sorted    # as printed: last met, first in the list
    assert nk == 2 and k_lit[14] == 1 and k_lit[9] == 1 and k_lit.sum() == 2
    # brute force: simulate the printed loop with a Python list on random inputs
    for _ in range(200):
        n = int(RNG.integers(1, 12))
        sw = RNG.uniform(-10, 60, n).round(1); sa = RNG.uniform(-10, 60, n).round(1)
        mw = RNG.choice([1e-6, 1e-6, 1e-6, 5e-4], n); ma = RNG.choice([1e-3, 1e-3, 1e-3, 1e-3, 9e-2], n)
        base = _py_rank(list(sw), list(mw), list(sa), list(ma))
        mean_w, mean_a = sum(mw) / n, sum(ma) / n
        sev = [max(mw[i] / mean_w, ma[i] / mean_a) for i in range(n)]
        lst = [i for i in base if not sev[i] > 5.0]      # L_sqnr: the non-outliers by ascending score
        for i in range(n):                               # the printed loop
            if sev[i] > 5.0:
                lst.insert(0, i)
        got, _, _ = oracle.rank_layers(sw, mw, sa, ma, outlier_order=1)
        assert got.tolist() == lst
        gf, _, _ = oracle.rank_layers_fused(sw, mw, sa, ma, None, outlier_order=1)
        assert gf.tolist() == lst


def test_rank_degenerate_variants_of_the_ablation():
    n = 12
    sw = RNG.uniform(20, 50, n); sa = RNG.uniform(20, 50, n)
    ones = np.ones(n)
    # activation gain 0 and no outliers: argsort of the weight-SQNR deltas
    order, _, _ = oracle.rank_layers(sw, ones, sa, ones, a_gain=0.0, w_gain=1.0)
    d = np.concatenate([[0.0], np.diff(sw)])
    assert order.tolist() == np.argsort(d, kind="stable").tolist()
    # feeding cumulative sums turns deltas back into raw SQNR: Weight-SQNR-Order baseline
    csw = np.cumsum(sw)
    order, _, _ = oracle.rank_layers(csw, ones, sa, ones, a_gain=0.0, w_gain=1.0, cap_db=1e9)
    expect = np.argsort(np.concatenate([[0.0], sw[1:]]), kind="stable").tolist()
    assert order.tolist() == expect
    # positions stretch the denominator
    pos = np.cumsum(RNG.integers(1, 4, n)).astype(float)
    order, _, _ = oracle.rank_layers(sw, ones, sa, ones, pos=pos)
    assert order.tolist() == _py_rank(list(sw), list(ones), list(sa), list(ones), list(pos))


def test_rank_matches_library_sort_on_random_inputs_and_is_a_permutation():
    for trial in range(300):
        n = int(RNG.integers(1, 9))
        sw = RNG.uniform(-10, 60, n).round(1)          # rounding provokes ties
        sa = RNG.uniform(-10, 60, n).round(1)
        mw = RNG.choice([0.0, 1e-6, 1e-5, 3e-4], n)
        ma = RNG.choice([1e-3, 2e-3, 9e-2], n)
        if trial % 7 == 0:
            sw[RNG.integers(0, n)] = math.inf          # zero-noise layer, clamped to the cap
        order, keep, nk = oracle.rank_layers(sw, mw, sa, ma)
        assert sorted(order.tolist()) == list(range(n))
        assert order.tolist() == _py_rank(list(sw), list(mw), list(sa), list(ma))
        assert nk == 0 and not keep.any()


def test_select_by_bops_rate_against_prefix_enumeration():
    for _ in range(200):
        n = int(RNG.integers(1, 9))
        sw = RNG.uniform(20, 50, n); sa = RNG.uniform(20, 50, n)
        macs = RNG.integers(0, 1000, n).astype(np.uint64)
        rate = int(RNG.integers(0, 10001))
        order, keep, nk = oracle.rank_layers(sw, np.ones(n), sa, np.ones(n), macs=macs,
                                             select_mode=1, rate_permyriad=rate)
        total = int(macs.sum())
        best = 0
        for k in range(n + 1):                         # every prefix, exact rationals
            q = total - sum(int(macs[i]) for i in order[:k])
            ok = Fraction(q * 10000) >= Fraction(rate * total)
            if ok:
                best = k
            else:
                break                                  # the rate only falls as the prefix grows
        assert nk == best
        assert keep.sum() == nk and all(keep[i] for i in order[:nk])
    # 0 % keeps everything in FP32, 100 % quantizes every layer that has work
    order, keep, nk = oracle.rank_layers([30, 20], [1, 1], [30, 20], [1, 1], macs=[5, 5],
                                         select_mode=1, rate_permyriad=0)
    assert nk == 2
    order, keep, nk = oracle.rank_layers([30, 20], [1, 1], [30, 20], [1, 1], macs=[5, 5],
                                         select_mode=1, rate_permyriad=10000)
    assert nk == 0
    order, keep, nk = oracle.rank_layers([30, 20], [1, 1], [30, 20], [1, 1], macs=[5, 5],
                                         select_mode=1, rate_permyriad=5000)
    assert nk == 1 and keep[order[0]] == 1


def test_rank_with_undefined_metrics_is_still_a_permutation():
    sw = [30.0, math.nan, 25.0, 40.0]
    sa = [30.0, 20.0, 25.0, 40.0]
    order, _, _ = oracle.rank_layers(sw, [1, 1, 1, 1], sa, [1, math.nan, 1, 1])
    # layers 1 and 2 have NaN deltas -> +inf score -> last, in layer order; a NaN MSE is no outlier
    assert order.tolist() == [0, 3, 1, 2]


# ---------------------------------------------------------------------------------- cosine
def test_cosine_closed_forms_and_library_dot_product():
    one = np.ones(1, np.float32); zero = np.zeros(1, np.float32)
    raw = lambda a, b: oracle.cosine(np.float32(a), np.float32(b), 1, 1, len(a), False, True,
                                     oracle.PAIR_RAW, one, one, zero)
    assert raw([1, 0], [0, 1]) == 0.0                       # orthogonal
    assert raw([1, 2, 3], [2, 4, 6]) == pytest.approx(1.0, abs=1e-15)    # parallel, any length
    assert raw([1, 2, 3], [-1, -2, -3]) == pytest.approx(-1.0, abs=1e-15)
    assert raw([1, 1], [1, 0]) == pytest.approx(1 / math.sqrt(2), abs=1e-15)
    assert raw([0, 0], [1, 2]) == 0.0 and raw([1, 2], [0, 0]) == 0.0     # a zero vector
    x = RNG.standard_normal(10_000).astype(np.float32)
    y = (x + 0.1 * RNG.standard_normal(10_000)).astype(np.float32)
    xd, yd = x.astype(np.float64), y.astype(np.float64)
    assert raw(x, y) == pytest.approx(xd @ yd / (np.linalg.norm(xd) * np.linalg.norm(yd)), abs=1e-14)
    assert raw(x, y) == pytest.approx(raw(y, x), abs=1e-15)              # symmetric
    # self mode: B is the dequantized tensor; on-grid data reproduces itself exactly
    d = 2.0 ** -7
    g = (np.arange(-127, 128) * d).astype(np.float32)
    r = _self(g)
    c1 = oracle.cosine(g, None, 1, 1, g.size, False, False, oracle.PAIR_SELF, r.step, r.inv, r.offset)
    assert c1 == pytest.approx(1.0, abs=1e-15)
    # and in general equals the dot-product form built from the codes
    r = _self(x)
    xh = r.codes.astype(np.float64) * float(r.step[0])
    got = oracle.cosine(x, None, 1, 1, x.size, False, False, oracle.PAIR_SELF, r.step, r.inv, r.offset)
    assert got == pytest.approx(xd @ xh / (np.linalg.norm(xd) * np.linalg.norm(xh)), abs=1e-14)
    # identity used by the GPU path: A.B = sig - sum(x e), |B|^2 = sig - 2 sum(x e) + sse
    e = xd - xh
    xe = float(xd @ e)
    assert got == pytest.approx((r.sig - xe) / math.sqrt(r.sig * (r.sig - 2 * xe + r.sse)), abs=1e-13)


# ------------------------------------------------------------------------ fusion-aware list
def test_fused_rank_hand_example_and_properties():
    NG = oracle.NO_GROUP
    sw = [40.0, 35.0, 37.0, 36.0, 42.0, 34.0]          # base order (see the hand-worked test): 5 1 0 2 3 4
    sa = [30.0, 31.0, 27.0, 30.0, 28.0, 29.0]
    one = [1.0] * 6
    base, _, _ = oracle.rank_layers(sw, one, sa, one)
    assert base.tolist() == [5, 1, 0, 2, 3, 4]
    # no groups at all, or everyone alone: the base list
    for fg in (None, [NG] * 6, [10, 11, 12, 13, 14, 15]):
        o, k, nk = oracle.rank_layers_fused(sw, one, sa, one, fg, keep_count=2)
        assert o.tolist() == base.tolist() and nk == 2 and k.tolist() == [0, 1, 0, 0, 0, 1]
    # layers 4 and 5 fuse (say conv + relu): 4 is pulled up beside 5, in layer order
    fg = [NG, NG, NG, NG, 7, 7]
    o, k, nk = oracle.rank_layers_fused(sw, one, sa, one, fg, keep_count=2)
    assert o.tolist() == [4, 5, 1, 0, 2, 3] and nk == 2 and k.tolist() == [0, 0, 0, 0, 1, 1]
    # a cut that would split the group keeps neither member
    o, k, nk = oracle.rank_layers_fused(sw, one, sa, one, fg, keep_count=1)
    assert nk == 0 and not k.any()
    o, k, nk = oracle.rank_layers_fused(sw, one, sa, one, fg, keep_count=3)
    assert nk == 3 and k.tolist() == [0, 1, 0, 0, 1, 1]
    # two groups: ordered by their best-ranked member (group {0,3} via layer 0 at base place 2,
    # group {1,2} via layer 1 at base place 1)
    fg = [3, 9, 9, 3, NG, NG]
    o, _, _ = oracle.rank_layers_fused(sw, one, sa, one, fg)
    assert o.tolist() == [5, 1, 2, 0, 3, 4]


def test_fused_rank_random_against_python_walk():
    NG = oracle.NO_GROUP
    for trial in range(200):
        n = int(RNG.integers(1, 12))
        sw = RNG.uniform(10, 60, n).round(1); sa = RNG.uniform(10, 60, n).round(1)
        mw = RNG.choice([1e-6, 1e-5, 3e-4], n); ma = RNG.choice([1e-3, 2e-3, 9e-2], n)
        fg = RNG.choice([NG, NG, 1, 2, 3], n).astype(np.uint32)
        macs = RNG.integers(0, 1000, n).astype(np.uint64)
        rate = int(RNG.integers(0, 10001)); kc = int(RNG.integers(0, n + 2)); mode = trial % 2
        base, _, _ = oracle.rank_layers(sw, mw, sa, ma)
        o, k, nk = oracle.rank_layers_fused(sw, mw, sa, ma, fg, macs=macs, select_mode=mode,
                                            keep_count=kc, rate_permyriad=rate)
        exp, seen = [], set()
        for l in base.tolist():
            if l in seen:
                continue
            members = [l] if fg[l] == NG else [m for m in range(n) if fg[m] == fg[l]]
            exp += members; seen.update(members)
        assert o.tolist() == exp and sorted(exp) == list(range(n))
        # selection: enumerate group boundaries
        bounds, j = [0], 0
        while j < n:
            e = j + 1
            while fg[exp[j]] != NG and e < n and fg[exp[e]] == fg[exp[j]]:
                e += 1
            bounds.append(e); j = e
        total = int(macs.sum()); best = 0
        for b in bounds[1:]:
            if mode == 0:
                ok = b <= kc
            else:
                q = total - sum(int(macs[i]) for i in exp[:b])
                ok = Fraction(q * 10000) >= Fraction(rate * total)
            if ok:
                best = b
            else:
                break
        assert nk == best and k.sum() == nk and all(k[i] for i in exp[:nk])


# ------------------------------------------------------------------------------- bit widths
@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8, 12, 16])
def test_bit_width_levels_on_grid_and_sqnr_closed_form(bits):
    qs, qa = 2 ** (bits - 1) - 1, 2 ** bits - 1               # Eq. 4's 2^(b-1)-1 and Eq. 2's N-1
    d = 2.0 ** -10
    k = np.arange(-qs, qs + 1)
    r = oracle.sweep_tensor((k * d).astype(np.float32), None, 1, 1, k.size, False, False,
                            want_codes=bits <= 8, bits=bits)
    assert r.step[0] == np.float32(d) and r.sse == 0.0 and r.sqnr_db == math.inf
    if bits <= 8:
        np.testing.assert_array_equal(r.codes, k.astype(np.int8))
    ka = np.arange(0, qa + 1)
    r = oracle.sweep_tensor((ka * d + 0.5).astype(np.float32), None, 1, 1, ka.size, False, True, bits=bits)
    assert r.step[0] == np.float32(d) and r.offset[0] == 0.5 and r.sse == 0.0
    # full-range uniform data: SQNR = 20 log10(2 qmax) symmetric, 10 log10(4 qmax^2) affine on [0,R]
    u = np.random.default_rng(bits).random(1 << 20)
    r = oracle.sweep_tensor(((2 * u - 1) * 3).astype(np.float32), None, 1, 1, u.size, False, False, bits=bits)
    assert r.sqnr_db == pytest.approx(20 * math.log10(2 * qs), abs=0.05)
    assert r.mse == pytest.approx(float(r.step[0]) ** 2 / 12, rel=2e-2 if bits > 2 else 0.2)
    if bits <= 12:      # beyond that the binary32 inputs themselves are coarser than the grid
        r = oracle.sweep_tensor((u * 5).astype(np.float32), None, 1, 1, u.size, False, True, bits=bits)
        assert r.sqnr_db == pytest.approx(10 * math.log10(4 * qa ** 2), abs=0.05)


def test_eight_bit_entry_points_are_the_bits_8_case():
    x = RNG.standard_normal(5000).astype(np.float32)
    a = oracle.sweep_tensor(x, None, 1, 1, 5000, False, True, want_codes=True)
    b = oracle.sweep_tensor(x, None, 1, 1, 5000, False, True, want_codes=True, bits=8)
    assert a.sse == b.sse and np.array_equal(a.codes, b.codes) and a.step[0] == b.step[0]
    c = oracle.sweep_tensor(x, None, 1, 1, 5000, False, True, bits=4)
    assert c.step[0] == np.float32(np.float32(a.gmax[0] - a.gmin[0]) / np.float32(15))
    assert c.mse > 200 * a.mse            # 4 fewer bits: about 2^8 = 256 times the noise power


# ------------------------------------------------------------------- integer zero point (scheme 2)
ZP = 2


def _zp(x, percentile=None, bits=8, y=None):
    x = np.asarray(x, np.float32)
    return oracle.sweep_tensor(x, y, 1, 1, x.size, False, ZP, percentile, want_codes=True, bits=bits)


def test_zero_point_represents_zero_exactly_and_widens_the_range():
    x = np.concatenate([np.zeros(50), RNG.uniform(-0.37, 1.91, 5000)]).astype(np.float32)
    r = _zp(x)
    z = int(r.offset[0])
    assert 0 < z < 255 and float(r.offset[0]) == z             # an integer, stored in the offset slot
    assert (r.codes[:50] == z).all()                           # x = 0 -> code z -> dequantized 0
    d = np.float32(r.gmax[0] - r.gmin[0])
    assert r.step[0] == d / np.float32(255) and r.inv[0] == np.float32(255) / d
    assert z == int(np.rint(np.float32(-r.gmin[0]) / r.step[0]))
    # an all-positive tensor: the range is widened down to 0, so z = 0 and step = max / 255
    pos = RNG.uniform(2.0, 5.0, 1000).astype(np.float32)
    r = _zp(pos)
    assert r.offset[0] == 0.0 and r.step[0] == np.float32(pos.max()) / np.float32(255) and r.codes.min() >= 102
    neg = -pos
    r = _zp(neg)
    assert r.offset[0] == 255.0 and r.codes.max() <= 153
    r = _zp(np.zeros(10))
    assert r.step[0] == 1.0 and r.offset[0] == 0.0 and r.sse == 0.0


def test_zero_point_equals_real_offset_when_the_minimum_is_on_the_grid():
    d = 2.0 ** -6
    x = (RNG.integers(-64, 192, 4000) * d + RNG.uniform(-0.4, 0.4, 4000) * d).astype(np.float32)
    x = np.clip(x, np.float32(-64 * d), np.float32(191 * d))
    x[0], x[1] = -64 * d, 191 * d                               # lo = -64 step, hi - lo = 255 step
    a = oracle.sweep_tensor(x, None, 1, 1, x.size, False, True, want_codes=True)
    b = _zp(x)
    assert a.step[0] == b.step[0] == np.float32(d) and b.offset[0] == 64.0 and a.offset[0] == np.float32(-64 * d)
    np.testing.assert_array_equal(a.codes, b.codes)
    assert b.sse == pytest.approx(a.sse, rel=1e-12)


def test_zero_point_against_library_quantizer_and_fractions():
    import torch
    x = (RNG.standard_normal(200_000) * 0.8 + 0.3).astype(np.float32)
    r = _zp(x)
    z = int(r.offset[0])
    qt = torch.quantize_per_tensor(torch.from_numpy(x), float(r.step[0]), z, torch.quint8).int_repr().numpy()
    diff = qt != r.codes
    assert diff.mean() < 1e-4 and np.abs(qt.astype(int) - r.codes.astype(int)).max() <= 1
    step = Fraction(float(r.step[0]))
    sse = Fraction(0)
    for v, q in zip(x[:300], r.codes[:300]):
        e = Fraction(float(v)) - (int(q) - z) * step
        assert abs(e) <= step / 2 + Fraction(1, 10 ** 6) or q in (0, 255)
        sse += e * e
    part = oracle.quant_metrics(x[:300], None, 1, 1, 300, False, ZP, oracle.PAIR_SELF, r.step, r.inv, r.offset)
    assert part["sse"] == pytest.approx(float(sse), rel=1e-14)
    # bit widths and saturation
    r4 = _zp(x, bits=4)
    assert r4.codes.max() == 15 and r4.codes.min() == 0 and 0 <= r4.offset[0] <= 15
    rc = _zp(np.concatenate([x, [40.0, -40.0]]), percentile=0.999)
    assert rc.codes[-2] == 255 and rc.codes[-1] == 0


# ------------------------------------------------------------------------------ KL divergence
def _kl_raw(a, b, A):
    one = np.ones(1, np.float32); zero = np.zeros(1, np.float32)
    a = np.float32(a); b = np.float32(b)
    return oracle.kl_divergence(a, b, 1, 1, a.size, False, True, oracle.PAIR_RAW, one, one, zero, A)


def test_kl_closed_forms_and_scipy():
    from scipy.special import rel_entr
    x = RNG.uniform(-4, 4, 50_000).astype(np.float32)
    kl, hp, hq = _kl_raw(x, x, 4.0)
    assert kl == 0.0 and np.array_equal(hp, hq) and hp.sum() == x.size        # identical -> 0
    kl, hp, hq = _kl_raw(x, -x, 4.0)
    assert kl == 0.0                                                          # |.| is what is binned
    y = (x * 0.5).astype(np.float32)                                          # mass moves to the lower half
    kl, hp, hq = _kl_raw(x, y, 4.0)
    assert hq[64:].sum() == 0 and hq.sum() == hp.sum() == x.size
    p = (hp + 1.0) / (x.size + 128); qq = (hq + 1.0) / (x.size + 128)
    assert kl == pytest.approx(float(rel_entr(p, qq).sum()), rel=1e-12) and kl > 0.5
    kl_rev, _, _ = _kl_raw(y, x, 4.0)
    assert kl_rev != pytest.approx(kl, rel=1e-3)                              # not symmetric
    # bins: planted centres with a power-of-two range are exact
    j = np.arange(128)
    c = ((j + 0.5) * (8.0 / 128)).astype(np.float32)
    kl, hp, hq = _kl_raw(c, c[::-1].copy(), 8.0)
    assert (hp == 1).all() and (hq == 1).all() and kl == 0.0
    kl, hp, hq = _kl_raw(np.float32([8.0, 100.0, np.nan, 1.0]), np.float32([8.0, 8.0, 1.0, np.inf]), 8.0)
    assert hp.sum() == 2 and hp[127] == 2 and hq[127] == 2                    # beyond A -> last bin; non-finite skipped
    # two-bin closed form: P = (3+1, 1+1)/(4+128) on bins 0 and 127 ... checked through the formula
    kl, hp, hq = _kl_raw(np.float32([0.0, 0.0, 0.0, 8.0]), np.float32([0.0, 8.0, 8.0, 8.0]), 8.0)
    den = 4 + 128
    exp = (4 / den) * math.log(4 / 2) + (2 / den) * math.log(2 / 4)
    assert kl == pytest.approx(exp, rel=1e-13)


def test_kl_of_quantized_tensor_uses_the_dequantized_values():
    x = RNG.standard_normal(100_000).astype(np.float32)
    r = _self(x)
    A = float(r.gabsmax[0])
    kl, hp, hq = oracle.kl_divergence(x, None, 1, 1, x.size, False, False, oracle.PAIR_SELF,
                                      r.step, r.inv, r.offset, A)
    xh = (r.codes.astype(np.float32) * r.step[0]).astype(np.float32)          # fl(q * step), offset 0
    w = np.float32(128) / np.float32(A)
    bins = lambda v: np.minimum((np.abs(v) * w).astype(np.float32).astype(np.int64), 127)
    assert np.array_equal(hp, np.bincount(bins(x), minlength=128)) and np.array_equal(hq, np.bincount(bins(xh), minlength=128))
    assert 0 < kl < 0.05                                                      # 8 bits: close distributions
    kl4, _, _ = oracle.kl_divergence(x, None, 1, 1, x.size, False, False, oracle.PAIR_SELF,
                                     *oracle.qparams(False, r.gmin, r.gmax, r.gabsmax, bits=4), A, bits=4)
    assert kl4 > 5 * kl                                                       # coarser grid, further apart


# -------------------------------------------------------------------------- Conv+BN folding
def test_fold_batchnorm_identity_equivalence_and_float32_ops():
    c, k = 7, 33
    w = RNG.standard_normal((c, k)).astype(np.float32); b = RNG.standard_normal(c).astype(np.float32)
    one = np.ones(c, np.float32); zero = np.zeros(c, np.float32)
    a, cc = oracle.fold_batchnorm(w, b, one, zero, zero, one)           # identity normalisation
    assert np.array_equal(a, w) and np.array_equal(cc, b)
    gamma = RNG.uniform(0.5, 2, c).astype(np.float32); beta = RNG.standard_normal(c).astype(np.float32)
    mean = RNG.standard_normal(c).astype(np.float32); var = RNG.uniform(0.1, 3, c).astype(np.float32)
    a, cc = oracle.fold_batchnorm(w, b, gamma, beta, mean, var)
    # functional meaning (Eq. 10 = Eq. 11): BN(W x + B) == A x + C for any input x
    x = RNG.standard_normal(k)
    conv = w.astype(np.float64) @ x + b
    bn = gamma * (conv - mean) / np.sqrt(var.astype(np.float64)) + beta
    np.testing.assert_allclose(a.astype(np.float64) @ x + cc, bn, rtol=0, atol=5e-6)
    # the same sequence of correctly rounded binary32 operations in numpy
    s = gamma / np.sqrt(var)                                               # float32 sqrt and divide
    assert np.array_equal(a, s[:, None] * w)
    assert np.array_equal(cc, s * (b - mean) + beta)
    a0, c0 = oracle.fold_batchnorm(w, None, gamma, beta, mean, var)        # no conv bias
    assert np.array_equal(a0, a) and np.array_equal(c0, s * (zero - mean) + beta)


# ------------------------------------------------------------------- per-channel percentile clip
def test_group_histograms_equal_per_tensor_histograms_of_each_channel_slice():
    """Channel c of an [O][C][I] tensor, cut out with numpy indexing, calibrated on its own as a
    per-tensor tensor, must give channel c's histogram, clip and parameters: this catches a wrong
    stride, a wrong group's absmax and a clip applied to the wrong channel."""
    rng = np.random.default_rng(77)
    O, Cn, I = 3, 5, 257
    x = (rng.standard_normal((O, Cn, I)) * (10.0 ** np.arange(-2, 3))[None, :, None]).astype(np.float32)
    x[1, 2, 7] = np.inf                                     # skipped in channel 2 only
    x[:, 4, :] = np.maximum(x[:, 4, :], 0)                  # a post-ReLU channel
    for asym in (0, 1, 2):
        gmin, gmax, gabs, bad, hist, clip, step, inv, off, ghist, gclip = oracle.calibrate_tensor(
            x, O, Cn, I, True, asym, 0.97, group_percentile=True)
        assert hist is None and bad == 1 and clip == gabs.max()
        for c in range(Cn):
            xc = np.ascontiguousarray(x[:, c, :])
            r = oracle.calibrate_tensor(xc, 1, 1, O * I, False, asym, 0.97)
            assert np.array_equal(ghist[c], r[4]), c
            assert gclip[c] == r[5], c
            assert step[c] == r[6][0] and inv[c] == r[7][0] and off[c] == r[8][0], c
            assert int(ghist[c].sum()) == O * I - (1 if c == 2 else 0)


def test_group_percentile_closed_form_and_difference_from_the_tensor_level_clip():
    """Two channels with known staircases: channel 0 holds k/1000 for k = 1..1000, channel 1 holds
    100x that.  With p = 0.9 each channel's clip is the upper edge of the bin that holds its 900th
    value, i.e. ~0.9 of ITS absmax, while a tensor-level histogram would put all of channel 0 in
    the lowest bins and leave it unclipped."""
    k = np.arange(1, 1001, dtype=np.float64)
    x = np.stack([k / 1000.0, k / 10.0]).astype(np.float32).reshape(1, 2, 1000)
    out = oracle.calibrate_tensor(x, 1, 2, 1000, True, 0, 0.9, group_percentile=True)
    gabs, step, gclip = out[2], out[6], out[10]
    for c in range(2):
        A = float(gabs[c])
        kstar = int(np.floor(np.float32(np.float32(x[0, c, 899]) * np.float32(np.float32(2048.0) / np.float32(A)))))
        assert abs(float(gclip[c]) - (kstar + 1) * A / 2048.0) <= 1e-6 * A
        assert 0.9 * A <= float(gclip[c]) <= 0.9 * A + A / 2048.0 * 1.001
        assert step[c] == np.float32(gclip[c]) / np.float32(127.0)
    t = oracle.calibrate_tensor(x, 1, 2, 1000, True, 0, 0.9)           # one clip for the tensor
    assert float(t[5]) > float(gabs[0])                                 # channel 0 is not clipped by it
    assert t[6][0] == np.float32(gabs[0]) / np.float32(127.0)
    # p = 1 clips nothing; a per-tensor tensor ignores the flag
    full = oracle.calibrate_tensor(x, 1, 2, 1000, True, 0, 1.0, group_percentile=True)
    assert np.array_equal(full[10], gabs)
    a = oracle.calibrate_tensor(x, 1, 2, 1000, False, 1, 0.9, group_percentile=True)
    b = oracle.calibrate_tensor(x, 1, 2, 1000, False, 1, 0.9)
    assert a[5] == b[5] and np.array_equal(a[4], b[4]) and np.array_equal(a[6], b[6])
