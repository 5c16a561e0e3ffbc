/*
 * CPU oracle for the local-metric sensitivity sweep of QuantuneV2 (arXiv 2501.07161).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, single-threaded definition that the
 * CUDA library is compared against.  It shares no code, header, table or helper with the CUDA
 * path and must never be linked, imported or called by it.  Element loops are written out one
 * element at a time, in the order and notation of the paper; there is no blocking, fusion or
 * vectorisation.
 *
 * Floating point.  Metrics are evaluated in double (accumulated in long double).  The few
 * operations whose rounding decides an INTEGER result (a scale, a code, a histogram bin) are
 * defined in binary32 and are written through the fl_* helpers below, each of which computes one
 * correctly rounded binary32 operation (the double result of +,-,*,/ on two floats rounds to
 * the same float as a native binary32 operation, since 53 >= 2*24+2).
 *
 * Parity pins (tests/test_oracle_*.py): every function here is pinned to closed forms,
 * brute force or invariants; none is "parity unpinned" except where noted:
 *   - the gain pair (w_gain, a_gain) of the ranking score is a constant the paper never prints;
 *     the default 2:1 is this build's reading ("parity unpinned" for that constant only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define QV2O_BINS 2048

/* one correctly rounded binary32 operation each */
static float fl_sub(float a, float b) { return (float)((double)a - (double)b); }
static float fl_mul(float a, float b) { return (float)((double)a * (double)b); }
static float fl_div(float a, float b) { return (float)((double)a / (double)b); }

static int finite_f(float v) { return isfinite(v) ? 1 : 0; }

/* ---------------------------------------------------------------------------------------------
 * Ranges (calibration, step 1 of the paper's overview; operands of Eq. 2 and Eq. 4).
 * Tensor viewed as [outer][channels][inner]; group of element (o,c,i) is c (per channel) or 0.
 * min, max over the finite elements of the group; absmax = max(|min|, |max|).
 * Non-finite elements are counted and excluded.  A zero result is +0.  A group without a
 * finite element reports 0 for all three.
 * ------------------------------------------------------------------------------------------- */
void qv2o_ranges(const float *x, uint64_t outer, uint64_t channels, uint64_t inner,
                 int per_channel, float *gmin, float *gmax, float *gabsmax, uint64_t *nonfinite)
{
    uint64_t groups = per_channel ? channels : 1;
    uint8_t *seen = (uint8_t *)calloc(groups ? groups : 1, 1);
    uint64_t bad = 0;
    for (uint64_t o = 0; o < outer; ++o)
        for (uint64_t c = 0; c < channels; ++c)
            for (uint64_t i = 0; i < inner; ++i) {
                float v = x[(o * channels + c) * inner + i];
                uint64_t g = per_channel ? c : 0;
                if (!finite_f(v)) { ++bad; continue; }
                if (!seen[g]) { gmin[g] = v; gmax[g] = v; seen[g] = 1; }
                else {
                    if (v < gmin[g]) gmin[g] = v;
                    if (v > gmax[g]) gmax[g] = v;
                }
            }
    for (uint64_t g = 0; g < groups; ++g) {
        if (!seen[g]) { gmin[g] = 0.0f; gmax[g] = 0.0f; }
        if (gmin[g] == 0.0f) gmin[g] = 0.0f;     /* -0 -> +0 */
        if (gmax[g] == 0.0f) gmax[g] = 0.0f;
        float a = fabsf(gmin[g]), b = fabsf(gmax[g]);
        gabsmax[g] = a > b ? a : b;
    }
    *nonfinite = bad;
    free(seen);
}

/* ---------------------------------------------------------------------------------------------
 * |x| histogram (the paper's calibration stage records a histogram of each layer's value range;
 * bin count and domain are this build's reading: 2048 linear bins of |x| on [0, A], A = the
 * tensor's absmax).  w = fl(2048 / A); bin = min(2047, trunc(fl(|x| * w))).
 * A == 0 or a non-finite w puts every element in bin 0.  Non-finite elements are skipped.
 * ------------------------------------------------------------------------------------------- */
void qv2o_histogram(const float *x, uint64_t n, float A, uint64_t *hist)
{
    memset(hist, 0, QV2O_BINS * sizeof(uint64_t));
    float w = (A > 0.0f) ? fl_div((float)QV2O_BINS, A) : 0.0f;
    if (!finite_f(w)) w = 0.0f;
    for (uint64_t k = 0; k < n; ++k) {
        float v = x[k];
        if (!finite_f(v)) continue;
        float f = fl_mul(fabsf(v), w);
        uint32_t b = (f >= (float)QV2O_BINS) ? (uint32_t)(QV2O_BINS - 1) : (uint32_t)f; /* trunc */
        if (b > QV2O_BINS - 1) b = QV2O_BINS - 1;
        hist[b] += 1;
    }
}

/* Percentile clip from the histogram: T = clamp(ceil(p * Nf), 1, Nf) with Nf = sum(hist);
 * k* = first bin whose cumulative count reaches T; clip = upper edge of bin k*:
 * A when k* is the last bin, else fl((k*+1) * fl(A / 2048)).  An empty histogram gives A. */
float qv2o_percentile_clip(const uint64_t *hist, double p, float A)
{
    uint64_t nf = 0;
    for (int j = 0; j < QV2O_BINS; ++j) nf += hist[j];
    if (nf == 0) return A;
    double t = ceil(p * (double)nf);
    uint64_t T;
    if (!(t >= 1.0)) T = 1;
    else if (t >= (double)nf) T = nf;
    else T = (uint64_t)t;
    uint64_t cum = 0;
    int kstar = QV2O_BINS - 1;
    for (int j = 0; j < QV2O_BINS; ++j) {
        cum += hist[j];
        if (cum >= T) { kstar = j; break; }
    }
    if (kstar == QV2O_BINS - 1) return A;
    return fl_mul((float)(kstar + 1), fl_div(A, (float)QV2O_BINS));
}

/* Per-channel variant of the calibration histogram: one 2048-bin |x| histogram for EVERY
 * quantization group c of a tensor laid out [outer][channels][inner], on [0, A_c] with A_c the
 * group's own absmax, and from it one clip value per group (same percentile rule as above).
 * hist: channels * 2048 counts; clip: channels values.  The paper's calibration keeps one
 * histogram per layer; this is the finer-grained reading for per-channel quantizers. */
void qv2o_group_histograms(const float *x, uint64_t outer, uint64_t channels, uint64_t inner,
                           const float *gabsmax, double p, uint64_t *hist, float *clip)
{
    memset(hist, 0, channels * QV2O_BINS * sizeof(uint64_t));
    for (uint64_t c = 0; c < channels; ++c) {
        const float A = gabsmax[c];
        float w = (A > 0.0f) ? fl_div((float)QV2O_BINS, A) : 0.0f;
        if (!finite_f(w)) w = 0.0f;
        uint64_t *h = hist + c * QV2O_BINS;
        for (uint64_t o = 0; o < outer; ++o)
            for (uint64_t i = 0; i < inner; ++i) {
                float v = x[(o * channels + c) * inner + i];
                if (!finite_f(v)) continue;
                float f = fl_mul(fabsf(v), w);
                uint32_t b = (f >= (float)QV2O_BINS) ? (uint32_t)(QV2O_BINS - 1) : (uint32_t)f;
                h[b] += 1;
            }
        clip[c] = qv2o_percentile_clip(h, p, A);
    }
}

/* ---------------------------------------------------------------------------------------------
 * Quantization parameters per group.
 * Symmetric int8 (Eq. 4, read as the multiplier S = 127 / max|W|): R = absmax_g, or
 * min(absmax_g, clip) when use_clip; step = fl(R / 127), inv = fl(127 / R), offset = 0.
 * Asymmetric uint8 (Eq. 2): lo = min_g, hi = max_g (clipped to [-clip, clip] when use_clip);
 * d = fl(hi - lo); step = fl(d / 255), inv = fl(255 / d), offset = lo (the real-valued x_min of
 * Eq. 1 and Eq. 3, not an integer zero point).
 * Degenerate range (zero, or a reciprocal that is not finite): step = inv = 1.
 * Affine form with an INTEGER zero point (scheme 2; what an integer-only accelerator runs, the
 * target the paper's compiler extension names): the range is first widened to contain 0,
 * lo' = min(lo, 0), hi' = max(hi, 0); d = fl(hi' - lo'); step = fl(d / top), inv = fl(top / d);
 * z = clamp(rne(fl(-lo' / step)), 0, top); the offset slot then carries z.  Codes are
 * q = clamp(rne(fl(v * inv)) + z, 0, top) and the dequantized value is (q - z) * step, so that
 * 0 is represented exactly.
 * ------------------------------------------------------------------------------------------- */
/* Levels of a b-bit quantizer: Eq. 4's 2^(b-1) - 1 for the symmetric scheme (codes in
 * [-qmax, qmax]), Eq. 2's N - 1 with N = 2^b levels for the affine one (codes in [0, qmax]). */
static int32_t top_code(int asym, int bits) { return asym ? (1 << bits) - 1 : (1 << (bits - 1)) - 1; }

void qv2o_qparams_bits(int bits, int asym_u8, int use_clip, float clip, uint64_t groups,
                  const float *gmin, const float *gmax, const float *gabsmax,
                  float *step, float *inv, float *offset)
{
    const float top = (float)top_code(asym_u8, bits);      /* 127 or 255 for 8 bits */
    for (uint64_t g = 0; g < groups; ++g) {
        float s, r, off;
        if (!asym_u8) {
            float R = gabsmax[g];
            if (use_clip && clip < R) R = clip;
            s = fl_div(R, top);
            r = fl_div(top, R);
            off = 0.0f;
            if (!(R > 0.0f) || !finite_f(r) || !(s > 0.0f)) { s = 1.0f; r = 1.0f; }
        } else {
            float lo = gmin[g], hi = gmax[g];
            if (use_clip) {
                if (-clip > lo) lo = -clip;
                if (clip < hi) hi = clip;
            }
            if (asym_u8 == 2) {                  /* integer zero point: the range must hold 0 */
                if (lo > 0.0f) lo = 0.0f;
                if (hi < 0.0f) hi = 0.0f;
            }
            if (lo == 0.0f) lo = 0.0f;
            float d = fl_sub(hi, lo);
            s = fl_div(d, top);
            r = fl_div(top, d);
            off = lo;
            if (!(d > 0.0f) || !finite_f(r) || !(s > 0.0f)) { s = 1.0f; r = 1.0f; if (asym_u8 == 2) off = 0.0f; }
            else if (asym_u8 == 2) {
                double z = nearbyint((double)fl_div(-lo, s));
                if (!(z >= 0.0)) z = 0.0;
                if (z > (double)top) z = (double)top;
                off = (float)z;
            }
        }
        step[g] = s; inv[g] = r; offset[g] = off;
    }
}

/* The same parameters with one clip value per group (per-channel percentile calibration). */
void qv2o_qparams_gclip(int bits, int scheme, uint64_t groups, const float *gclip,
                        const float *gmin, const float *gmax, const float *gabsmax,
                        float *step, float *inv, float *offset)
{
    for (uint64_t g = 0; g < groups; ++g)
        qv2o_qparams_bits(bits, scheme, 1, gclip[g], 1, gmin + g, gmax + g, gabsmax + g,
                          step + g, inv + g, offset + g);
}

void qv2o_qparams(int asym_u8, int use_clip, float clip, uint64_t groups,
                  const float *gmin, const float *gmax, const float *gabsmax,
                  float *step, float *inv, float *offset)
{
    qv2o_qparams_bits(8, asym_u8, use_clip, clip, groups, gmin, gmax, gabsmax, step, inv, offset);
}

/* One code (Eq. 1 / Eq. 5): t = fl(fl(v - offset) * inv); q = clamp(rne(t), qmin, qmax), the
 * rounding being to nearest with ties to even and the clamp saturating. */
static int32_t quant_code(float v, float inv, float offset, int32_t qmin, int32_t qmax)
{
    float t = fl_mul(fl_sub(v, offset), inv);
    if (isnan(t)) return qmin;
    double r = nearbyint((double)t);       /* default rounding mode: ties to even */
    if (r < (double)qmin) return qmin;
    if (r > (double)qmax) return qmax;
    return (int32_t)r;
}

/* One code with an integer zero point z: q = clamp(rne(fl(v * inv)) + z, 0, qmax). */
static int32_t quant_code_zp(float v, float inv, int32_t z, int32_t qmax)
{
    float t = fl_mul(v, inv);
    if (isnan(t)) return 0;
    double r = nearbyint((double)t) + (double)z;
    if (r < 0.0) return 0;
    if (r > (double)qmax) return qmax;
    return (int32_t)r;
}

/* ---------------------------------------------------------------------------------------------
 * Fake-quantize and reduce the error (Eq. 1, 3, 5 for the codes and their dequantized values,
 * Eq. 6 for SQNR, Eq. 7 for MSE).
 *   pair_mode 0 (self):     v = x,  xhat = q(x)*step + offset,  e = x - xhat     (weights)
 *   pair_mode 1 (requant):  v = y,  yhat = q(y)*step + offset,  e = x - yhat     (activations:
 *                           reference pass x against the quantized pass y put on x's grid)
 *   pair_mode 2 (raw):      e = x - y, no codes
 * SSE = sum e^2 (P_noise), SIG = sum x^2 (P_signal, always the reference tensor);
 * MSE = SSE / N;  SQNR = 10 log10(SIG / SSE), +inf when SSE == 0, -inf when SIG == 0 < SSE.
 * Metrics are per tensor even when the parameters are per channel.
 * codes (nullable) receives one byte per element: int8 for the symmetric scheme, uint8 else
 * (the low byte of the code; meaningful for bit widths up to 8).
 * ------------------------------------------------------------------------------------------- */
void qv2o_quant_metrics_bits(int bits, const float *x, const float *y,
                        uint64_t outer, uint64_t channels, uint64_t inner, int per_channel,
                        int asym_u8, int pair_mode,
                        const float *step, const float *inv, const float *offset,
                        uint8_t *codes, double *sse_out, double *sig_out,
                        double *mse_out, double *sqnr_out)
{
    int32_t qmax = top_code(asym_u8, bits), qmin = asym_u8 ? 0 : -qmax;
    long double sse = 0.0L, sig = 0.0L;
    uint64_t n = outer * channels * inner;
    for (uint64_t o = 0; o < outer; ++o)
        for (uint64_t c = 0; c < channels; ++c)
            for (uint64_t i = 0; i < inner; ++i) {
                uint64_t k = (o * channels + c) * inner + i;
                uint64_t g = per_channel ? c : 0;
                double xr = (double)x[k], e;
                if (pair_mode == 2) {
                    e = xr - (double)y[k];
                } else {
                    float v = (pair_mode == 1) ? y[k] : x[k];
                    int32_t q;
                    double deq;
                    if (asym_u8 == 2) {
                        int32_t z = (int32_t)offset[g];
                        q = quant_code_zp(v, inv[g], z, qmax);
                        deq = (double)(q - z) * (double)step[g];
                    } else {
                        q = quant_code(v, inv[g], offset[g], qmin, qmax);
                        deq = (double)q * (double)step[g] + (double)offset[g];
                    }
                    e = xr - deq;
                    if (codes) codes[k] = (uint8_t)(q & 0xFF);
                }
                sse += (long double)e * (long double)e;
                sig += (long double)xr * (long double)xr;
            }
    double dsse = (double)sse, dsig = (double)sig;
    *sse_out = dsse;
    *sig_out = dsig;
    *mse_out = n ? dsse / (double)n : 0.0;
    if (dsse == 0.0) *sqnr_out = INFINITY;
    else if (dsig == 0.0) *sqnr_out = -INFINITY;
    else *sqnr_out = 10.0 * log10(dsig / dsse);
}

void qv2o_quant_metrics(const float *x, const float *y,
                        uint64_t outer, uint64_t channels, uint64_t inner, int per_channel,
                        int asym_u8, int pair_mode,
                        const float *step, const float *inv, const float *offset,
                        uint8_t *codes, double *sse_out, double *sig_out,
                        double *mse_out, double *sqnr_out)
{
    qv2o_quant_metrics_bits(8, x, y, outer, channels, inner, per_channel, asym_u8, pair_mode, step, inv,
                            offset, codes, sse_out, sig_out, mse_out, sqnr_out);
}

/* ---------------------------------------------------------------------------------------------
 * Cosine similarity (Eq. 8): A.B / (|A| |B|) with A the reference tensor x and B the tensor it is
 * compared with -- the dequantized copy of x (pair_mode 0), the dequantized re-quantization of y
 * (pair_mode 1) or y itself (pair_mode 2).  Written straight from the definition, three sums in
 * long double.  A zero vector has no direction: the result is then 0.
 * ------------------------------------------------------------------------------------------- */
double qv2o_cosine_bits(int bits, const float *x, const float *y,
                   uint64_t outer, uint64_t channels, uint64_t inner, int per_channel,
                   int asym_u8, int pair_mode,
                   const float *step, const float *inv, const float *offset)
{
    int32_t qmax = top_code(asym_u8, bits), qmin = asym_u8 ? 0 : -qmax;
    long double ab = 0.0L, aa = 0.0L, bb = 0.0L;
    for (uint64_t o = 0; o < outer; ++o)
        for (uint64_t c = 0; c < channels; ++c)
            for (uint64_t i = 0; i < inner; ++i) {
                uint64_t k = (o * channels + c) * inner + i;
                uint64_t g = per_channel ? c : 0;
                long double a = (long double)x[k], b;
                if (pair_mode == 2) {
                    b = (long double)y[k];
                } else {
                    float v = (pair_mode == 1) ? y[k] : x[k];
                    if (asym_u8 == 2) {
                        int32_t z = (int32_t)offset[g];
                        int32_t q = quant_code_zp(v, inv[g], z, qmax);
                        b = (long double)(q - z) * (long double)step[g];
                    } else {
                        int32_t q = quant_code(v, inv[g], offset[g], qmin, qmax);
                        b = (long double)q * (long double)step[g] + (long double)offset[g];
                    }
                }
                ab += a * b; aa += a * a; bb += b * b;
            }
    long double den = sqrtl(aa) * sqrtl(bb);
    return den > 0.0L ? (double)(ab / den) : 0.0;
}

double qv2o_cosine(const float *x, const float *y,
                   uint64_t outer, uint64_t channels, uint64_t inner, int per_channel,
                   int asym_u8, int pair_mode,
                   const float *step, const float *inv, const float *offset)
{
    return qv2o_cosine_bits(8, x, y, outer, channels, inner, per_channel, asym_u8, pair_mode, step, inv, offset);
}

/* ---------------------------------------------------------------------------------------------
 * KL divergence (Eq. 9): sum_x P(x) log(P(x) / Q(x)), P the distribution of the original tensor's
 * values and Q that of the tensor it is compared with (dequantized x, dequantized re-quantized y,
 * or y).  The paper gives no discretisation; the reading taken here: both tensors are binned on
 * the same QV2O_KL_BINS = 128 linear bins of |value| over [0, A], A the reference tensor's
 * absmax (values beyond A fall in the last bin); w = fl(128 / A), bin(v) = min(127,
 * trunc(fl(|v| * w))); counts get add-one smoothing, P_j = (hp_j + 1) / (N + 128), same for Q;
 * the result is in nats.  The compared value is formed in binary32 so that its bin is a fixed
 * function of the inputs: b = fl(fl(q * step) + offset) (offset 0 adds nothing; with an integer
 * zero point b = fl((q - z) * step)); in raw mode b = y.  Non-finite values are skipped.
 * hp / hq (nullable) receive the two 128-bin histograms.
 * ------------------------------------------------------------------------------------------- */
#define QV2O_KL_BINS 128

static uint32_t kl_bin(float v, float w)
{
    float f = fl_mul(fabsf(v), w);
    if (!(f < (float)QV2O_KL_BINS)) return QV2O_KL_BINS - 1;
    return (uint32_t)f;
}

double qv2o_kl_bits(int bits, const float *x, const float *y,
                    uint64_t outer, uint64_t channels, uint64_t inner, int per_channel,
                    int asym_u8, int pair_mode,
                    const float *step, const float *inv, const float *offset, float A,
                    uint64_t *hp_out, uint64_t *hq_out)
{
    int32_t qmax = top_code(asym_u8, bits), qmin = asym_u8 ? 0 : -qmax;
    uint64_t hp[QV2O_KL_BINS] = {0}, hq[QV2O_KL_BINS] = {0};
    float w = (A > 0.0f) ? fl_div((float)QV2O_KL_BINS, A) : 0.0f;
    if (!finite_f(w)) w = 0.0f;
    uint64_t n = 0;
    for (uint64_t o = 0; o < outer; ++o)
        for (uint64_t c = 0; c < channels; ++c)
            for (uint64_t i = 0; i < inner; ++i) {
                uint64_t k = (o * channels + c) * inner + i;
                uint64_t g = per_channel ? c : 0;
                float b;
                if (pair_mode == 2) {
                    b = y[k];
                } else {
                    float v = (pair_mode == 1) ? y[k] : x[k];
                    if (asym_u8 == 2) {
                        int32_t z = (int32_t)offset[g];
                        int32_t q = quant_code_zp(v, inv[g], z, qmax);
                        b = fl_mul((float)(q - z), step[g]);
                    } else {
                        int32_t q = quant_code(v, inv[g], offset[g], qmin, qmax);
                        b = fl_mul((float)q, step[g]);
                        b = (float)((double)b + (double)offset[g]);
                    }
                }
                if (!finite_f(x[k]) || !finite_f(b)) continue;
                hp[kl_bin(x[k], w)] += 1;
                hq[kl_bin(b, w)] += 1;
                ++n;
            }
    double kl = 0.0, den = (double)n + (double)QV2O_KL_BINS;
    for (int j = 0; j < QV2O_KL_BINS; ++j) {
        double p = ((double)hp[j] + 1.0) / den, q = ((double)hq[j] + 1.0) / den;
        kl += p * log(p / q);
    }
    if (hp_out) memcpy(hp_out, hp, sizeof(hp));
    if (hq_out) memcpy(hq_out, hq, sizeof(hq));
    return kl;
}

/* ---------------------------------------------------------------------------------------------
 * Sensitivity list (Algorithm 2 with RankLayersBySensitivity, Eq. 16 for the SQNR delta) and
 * the FP32-kept set for a requested quantization level (Eq. 17, normalised).
 *  1. every SQNR is clamped to [-cap, cap].
 *  2. delta_0 = 0; delta_n = (sqnr[n] - sqnr[n-1]) / (pos[n] - pos[n-1])  (pos defaults to n).
 *  3. score_n = w_gain * dw_n + a_gain * da_n  (the weighted sum of the two delta lists).
 *  4. r_n = max(mse_w[n] / mean(mse_w), mse_a[n] / mean(mse_a)), a zero mean contributing 0;
 *     layers with r_n > mse_factor (5 in the paper) go to the top, most severe first (or, on
 *     request, in the order the printed pseudo-code produces: see qv2o_rank_ex).
 *  5. the remaining layers follow in ascending score (smaller delta = noise grew = more
 *     sensitive); ties keep layer order.  A NaN score counts as +inf, a NaN severity as 0 (the
 *     paper does not say what an undefined metric does; this keeps the list a permutation).
 *  6. select_mode 0: the first keep_count entries stay FP32.  select_mode 1: the longest prefix
 *     stays FP32 for which the MAC-weighted share of quantized layers is still
 *     >= rate_permyriad / 10000 (integer arithmetic).
 * Means are sums in layer order divided by n; all arithmetic is one double operation at a time.
 * ------------------------------------------------------------------------------------------- */
static double clampd(double v, double cap)
{
    if (v > cap) return cap;
    if (v < -cap) return -cap;
    return v;
}

/* outlier_order 0: MSE outliers most severe first (the reading this library takes by default).
 * outlier_order 1: Algorithm 2's RankLayersBySensitivity as printed: the layers are visited in
 * order and each outlier is inserted at the head of the list when it is met, so the outliers end
 * in reverse layer order. */
void qv2o_rank_ex(uint32_t n, const double *sqnr_w, const double *mse_w,
                  const double *sqnr_a, const double *mse_a,
                  const uint64_t *macs, const double *pos,
                  double w_gain, double a_gain, double mse_factor, double cap,
                  int select_mode, uint32_t keep_count, uint32_t rate_permyriad, int outlier_order,
                  uint32_t *order, uint8_t *keep, uint32_t *n_keep)
{
    if (n == 0) { *n_keep = 0; return; }
    double *score = (double *)malloc(n * sizeof(double));
    double *sev = (double *)malloc(n * sizeof(double));
    uint8_t *taken = (uint8_t *)calloc(n, 1);
    double sum_w = 0.0, sum_a = 0.0;
    for (uint32_t i = 0; i < n; ++i) { sum_w += mse_w[i]; sum_a += mse_a[i]; }
    double mean_w = sum_w / (double)n, mean_a = sum_a / (double)n;
    for (uint32_t i = 0; i < n; ++i) {
        double dw = 0.0, da = 0.0;
        if (i > 0) {
            double den = pos ? (pos[i] - pos[i - 1]) : 1.0;
            dw = (clampd(sqnr_w[i], cap) - clampd(sqnr_w[i - 1], cap)) / den;
            da = (clampd(sqnr_a[i], cap) - clampd(sqnr_a[i - 1], cap)) / den;
        }
        double tw = w_gain * dw;
        double ta = a_gain * da;
        score[i] = tw + ta;
        if (isnan(score[i])) score[i] = INFINITY;      /* an undefined score sorts last */
        double rw = (mean_w > 0.0) ? mse_w[i] / mean_w : 0.0;
        double ra = (mean_a > 0.0) ? mse_a[i] / mean_a : 0.0;
        sev[i] = rw > ra ? rw : ra;
        if (isnan(sev[i])) sev[i] = 0.0;               /* an undefined severity is no outlier */
    }
    /* selection sort, written for clarity: repeatedly take the best remaining layer */
    uint32_t filled = 0;
    if (outlier_order == 1) {                    /* each outlier goes to the head as it is met */
        for (uint32_t i = 0; i < n; ++i) {
            if (!(sev[i] > mse_factor)) continue;
            for (uint32_t k = filled; k > 0; --k) order[k] = order[k - 1];
            order[0] = i; taken[i] = 1; ++filled;
        }
    } else for (;;) {                            /* MSE outliers, most severe first */
        int best = -1;
        for (uint32_t i = 0; i < n; ++i)
            if (!taken[i] && sev[i] > mse_factor && (best < 0 || sev[i] > sev[best])) best = (int)i;
        if (best < 0) break;
        taken[best] = 1; order[filled++] = (uint32_t)best;
    }
    while (filled < n) {                         /* the rest, ascending score */
        int best = -1;
        for (uint32_t i = 0; i < n; ++i)
            if (!taken[i] && (best < 0 || score[i] < score[best])) best = (int)i;
        taken[best] = 1; order[filled++] = (uint32_t)best;
    }
    uint32_t nk = 0;
    if (select_mode == 0) {
        nk = keep_count < n ? keep_count : n;
    } else {
        unsigned __int128 total = 0;
        for (uint32_t i = 0; i < n; ++i) total += macs ? macs[i] : 1;
        unsigned __int128 kept = 0;
        nk = 0;
        for (uint32_t j = 0; j < n; ++j) {       /* grow the FP32 prefix while the rate holds */
            unsigned __int128 m = macs ? macs[order[j]] : 1;
            unsigned __int128 quantized = total - (kept + m);
            if (quantized * 10000 >= (unsigned __int128)rate_permyriad * total) { kept += m; nk = j + 1; }
            else break;
        }
    }
    for (uint32_t i = 0; i < n; ++i) keep[i] = 0;
    for (uint32_t j = 0; j < nk; ++j) keep[order[j]] = 1;
    *n_keep = nk;
    free(score); free(sev); free(taken);
}

void qv2o_rank(uint32_t n, const double *sqnr_w, const double *mse_w,
               const double *sqnr_a, const double *mse_a,
               const uint64_t *macs, const double *pos,
               double w_gain, double a_gain, double mse_factor, double cap,
               int select_mode, uint32_t keep_count, uint32_t rate_permyriad,
               uint32_t *order, uint8_t *keep, uint32_t *n_keep)
{
    qv2o_rank_ex(n, sqnr_w, mse_w, sqnr_a, mse_a, macs, pos, w_gain, a_gain, mse_factor, cap,
                 select_mode, keep_count, rate_permyriad, 0, order, keep, n_keep);
}

/* ---------------------------------------------------------------------------------------------
 * Fusion-aware sensitivity list.  The paper says only that fusion-capable operators (convolution,
 * batch normalisation, add, ReLU) may have their positions in the list adjusted so that they can
 * be fused and share one bit-width.  Reading taken here: fuse_group[i] names the fusion group of
 * layer i (QV2O_NO_GROUP = on its own).  The base list is qv2o_rank's; walking it from the top,
 * the first time a member of a group is met the whole group is emitted at that place in layer
 * order, and later members are skipped.  The FP32-kept prefix never splits a group: by count it
 * is the longest run of whole groups with at most keep_count layers; by rate it grows group by
 * group while the MAC-weighted share of still-quantized layers is >= rate_permyriad / 10000.
 * ------------------------------------------------------------------------------------------- */
#define QV2O_NO_GROUP 0xFFFFFFFFu

void qv2o_rank_fused_ex(uint32_t n, const double *sqnr_w, const double *mse_w,
                        const double *sqnr_a, const double *mse_a,
                        const uint64_t *macs, const double *pos, const uint32_t *fuse_group,
                        double w_gain, double a_gain, double mse_factor, double cap,
                        int select_mode, uint32_t keep_count, uint32_t rate_permyriad, int outlier_order,
                        uint32_t *order, uint8_t *keep, uint32_t *n_keep)
{
    if (n == 0) { *n_keep = 0; return; }
    uint32_t *base = (uint32_t *)malloc(n * sizeof(uint32_t));
    uint8_t *tmp_keep = (uint8_t *)malloc(n);
    uint32_t tmp_nk;
    qv2o_rank_ex(n, sqnr_w, mse_w, sqnr_a, mse_a, macs, pos, w_gain, a_gain, mse_factor, cap,
                 0, 0, 0, outlier_order, base, tmp_keep, &tmp_nk);
    uint8_t *done = (uint8_t *)calloc(n, 1);
    uint32_t filled = 0;
    for (uint32_t j = 0; j < n; ++j) {
        uint32_t l = base[j];
        if (done[l]) continue;
        uint32_t g = fuse_group ? fuse_group[l] : QV2O_NO_GROUP;
        if (g == QV2O_NO_GROUP) { order[filled++] = l; done[l] = 1; continue; }
        for (uint32_t m = 0; m < n; ++m)            /* the whole group, in layer order */
            if (fuse_group[m] == g) { order[filled++] = m; done[m] = 1; }
    }
    unsigned __int128 total = 0, kept = 0;
    for (uint32_t i = 0; i < n; ++i) total += macs ? macs[i] : 1;
    uint32_t nk = 0, j = 0;
    while (j < n) {                                  /* one whole group at a time */
        uint32_t g = fuse_group ? fuse_group[order[j]] : QV2O_NO_GROUP;
        uint32_t e = j + 1;
        if (g != QV2O_NO_GROUP) while (e < n && fuse_group[order[e]] == g) ++e;
        if (select_mode == 0) {
            if (e <= keep_count) nk = e; else break;
        } else {
            unsigned __int128 m = 0;
            for (uint32_t k = j; k < e; ++k) m += macs ? macs[order[k]] : 1;
            unsigned __int128 quantized = total - (kept + m);
            if (quantized * 10000 >= (unsigned __int128)rate_permyriad * total) { kept += m; nk = e; }
            else break;
        }
        j = e;
    }
    for (uint32_t i = 0; i < n; ++i) keep[i] = 0;
    for (uint32_t k = 0; k < nk; ++k) keep[order[k]] = 1;
    *n_keep = nk;
    free(base); free(tmp_keep); free(done);
}

void qv2o_rank_fused(uint32_t n, const double *sqnr_w, const double *mse_w,
                     const double *sqnr_a, const double *mse_a,
                     const uint64_t *macs, const double *pos, const uint32_t *fuse_group,
                     double w_gain, double a_gain, double mse_factor, double cap,
                     int select_mode, uint32_t keep_count, uint32_t rate_permyriad,
                     uint32_t *order, uint8_t *keep, uint32_t *n_keep)
{
    qv2o_rank_fused_ex(n, sqnr_w, mse_w, sqnr_a, mse_a, macs, pos, fuse_group, w_gain, a_gain, mse_factor,
                       cap, select_mode, keep_count, rate_permyriad, 0, order, keep, n_keep);
}

/* ---------------------------------------------------------------------------------------------
 * Convolution + batch-normalisation folding (Eq. 10-12): A_c = gamma_c / sqrt(var_c) * W_c,
 * C_c = gamma_c (B_c - mean_c) / sqrt(var_c) + beta_c.  The outputs are binary32 tensors that feed
 * the sweep, so every operation is one binary32 rounding, in this order: r = sqrt(var),
 * s = gamma / r, A = s * W, C = (s * (B - mean)) + beta.  bias may be NULL (zeros).
 * ------------------------------------------------------------------------------------------- */
void qv2o_fold_batchnorm(const float *w, const float *bias, const float *gamma, const float *beta,
                         const float *mean, const float *var, uint64_t channels, uint64_t inner,
                         float *w_out, float *bias_out)
{
    for (uint64_t c = 0; c < channels; ++c) {
        float r = (float)sqrt((double)var[c]);          /* correctly rounded: 53 >= 2*24 + 2 */
        float s = fl_div(gamma[c], r);
        for (uint64_t k = 0; k < inner; ++k) w_out[c * inner + k] = fl_mul(s, w[c * inner + k]);
        if (bias_out) {
            float b = bias ? bias[c] : 0.0f;
            bias_out[c] = (float)((double)fl_mul(s, fl_sub(b, mean[c])) + (double)beta[c]);
        }
    }
}
