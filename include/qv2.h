/*
 * qv2 -- local-metric sensitivity sweep of QuantuneV2 (arXiv 2501.07161) on one NVIDIA B200.
 *
 * For every layer of a model the sweep calibrates quantization ranges over the weight tensor and
 * the captured activation tensor, fake-quantizes to 8 bit, reduces the quantization error to MSE
 * and SQNR, and finally scores, ranks and selects the layers that stay in FP32 (the paper's
 * "Sensitivity Analyzer", steps 1-4 of its overview and Algorithm 2).
 *
 * Conventions common to every call
 *   - Plain C ABI.  Every function returns an int status: QV2_OK (0) or a negative QV2_ERR_*.
 *     Nothing throws, aborts or traps on the device.
 *   - "device" pointers are CUDA global-memory addresses valid on the context's device, "host"
 *     pointers are ordinary process memory.  The caller owns every tensor and every output buffer;
 *     the library owns only the scratch inside qv2_ctx (tile tables and partial sums), grown on
 *     demand and released by qv2_destroy.
 *   - Calls enqueue work on the context's stream and return; outputs are valid once the caller has
 *     synchronised that stream.  Argument errors are found on the host before anything is
 *     launched.  Exceptions: a call whose descriptor set (the qv2_tensor_desc bytes) differs from
 *     the previous call's synchronises the stream once while it rebuilds its tile table -- the
 *     code pointers of qv2_quant_metrics are not part of that set -- and qv2_sweep_model_host
 *     and qv2_check_nonfinite synchronise before they return.  qv2_sync_count reports how often
 *     a context has done so.
 *   - Accumulators that must start at zero (range keys, counters, histograms, tickets) live in
 *     context scratch and are put back to zero by the code that consumes them, so a pass needs
 *     no clearing launch.  Partial results of a tensor are folded either by whichever thread
 *     block finishes the tensor last, found with an atomic counter, or by a small follow-up
 *     kernel (qv2_set_fold_mode); no block ever waits for another.
 *   - One context serves one stream; use it from one host thread at a time.
 *   - Tensors are fp32, contiguous, viewed as [outer][channels][inner]; element (o,c,i) lives at
 *     index (o*channels + c)*inner + i.  Weights: outer = 1, channels = C_out, inner = C_in/g*k*k.
 *     Activations: outer = batch, channels = C, inner = H*W.  The quantization group of an element
 *     is its channel c (QV2_PER_CHANNEL) or 0 (QV2_PER_TENSOR).  Per-group arrays hold the groups
 *     of descs[0], then those of descs[1], ...; qv2_group_count gives the total.
 *   - Non-finite input elements are counted into nonfinite[]; they are left out of ranges and
 *     histograms, and the metrics of a tensor that has any are unspecified.
 */
#ifndef QV2_H_
#define QV2_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QV2_HIST_BINS 2048

enum {
  QV2_OK = 0,
  QV2_ERR_ARG = -1,         /* bad enum value, inconsistent sizes, percentile outside [0,1] */
  QV2_ERR_NULL = -2,        /* a required pointer is NULL */
  QV2_ERR_ALIGN = -3,       /* a tensor pointer is not 4-byte aligned */
  QV2_ERR_SIZE = -4,        /* a size exceeds what the library supports (see each call) */
  QV2_ERR_NONFINITE = -5,   /* reported by qv2_sweep_model_host when an input held NaN or Inf */
  QV2_ERR_CUDA = -6,        /* a CUDA runtime call failed; see qv2_last_cuda_error */
  QV2_ERR_NOMEM = -7,       /* scratch allocation failed */
  QV2_ERR_UNSUPPORTED = -8  /* a combination the library does not implement */
};

enum { QV2_PER_TENSOR = 0, QV2_PER_CHANNEL = 1 };            /* granularity */
enum { QV2_SYM_I8 = 0, QV2_ASYM_U8 = 1, QV2_ASYM_U8_ZP = 2 }; /* scheme */
enum { QV2_ABSMAX = 0, QV2_MINMAX = 1, QV2_PERCENTILE = 2, QV2_PERCENTILE_GROUP = 3 }; /* range */
enum { QV2_PAIR_REQUANT = 0, QV2_PAIR_RAW = 1, QV2_STORE_CODES = 2 }; /* flags (bit 0: pair mode) */
enum { QV2_BY_COUNT = 0, QV2_BY_BOPS_RATE = 1 };             /* select_mode */
enum { QV2_OUTLIERS_BY_SEVERITY = 0, QV2_OUTLIERS_LITERAL = 1 }; /* outlier_order */
enum { QV2_SCHEDULE_PHASE_MAJOR = 0, QV2_SCHEDULE_L2_CHUNKED = 1, QV2_SCHEDULE_AUTO = 2 };
enum { QV2_FOLD_AUTO = 0, QV2_FOLD_FUSED = 1, QV2_FOLD_SEPARATE = 2 };
/* Code width other than 8 bits, OR-ed into qv2_tensor_desc.flags: QV2_BITS(b), 2 <= b <= 16.  The
 * largest code is 2^(b-1) - 1 for QV2_SYM_I8 (Eq. 4) and 2^b - 1 for QV2_ASYM_U8 (Eq. 2 with
 * N = 2^b levels); wherever this header says 127 or 255 read that value.  No QV2_BITS means 8.
 * QV2_STORE_CODES needs b <= 8 (codes are one byte), else QV2_ERR_UNSUPPORTED. */
/* Element type of the tensors x and y, OR-ed into flags.  The default is binary32.  With
 * QV2_IN_F16 / QV2_IN_BF16 the pointers x and y (declared const float* for the ABI) address
 * IEEE binary16 / bfloat16 data, 2-byte aligned; every value is widened exactly to binary32 and
 * all arithmetic is as documented for binary32, so the pass moves half the bytes.  Not accepted
 * by qv2_quant_metrics_noalloc. */
#define QV2_IN_F32 0u
#define QV2_IN_F16 (1u << 16)
#define QV2_IN_BF16 (2u << 16)
#define QV2_IN_MASK (3u << 16)
#define QV2_BITS(b) ((uint32_t)(b) << 8)
#define QV2_BITS_MASK 0xFF00u
#define QV2_DESC_BITS(flags) (((flags) & QV2_BITS_MASK) ? (((uint32_t)(flags) & QV2_BITS_MASK) >> 8) : 8u)

typedef struct qv2_ctx qv2_ctx;

/* One tensor of one layer. */
typedef struct {
  const float* x;        /* device (host for qv2_sweep_model_host); reference tensor; may be NULL
                            only when the tensor has no elements */
  const float* y;        /* nullable; the same tensor as produced by the quantized pass.  NULL
                            selects self mode (weights): the error is x against its own
                            dequantized copy.  Non-NULL selects pair mode (activations). */
  uint64_t outer, channels, inner;
  uint32_t granularity;  /* QV2_PER_TENSOR | QV2_PER_CHANNEL */
  uint32_t scheme;       /* QV2_SYM_I8: codes in [-127,127], offset 0.
                            QV2_ASYM_U8: codes in [0,255], real-valued offset = range minimum
                            QV2_ASYM_U8_ZP: codes in [0,255] with an integer zero point z (what an
                            integer-only accelerator runs): the range is widened to contain 0,
                            z = clamp(round(-lo/step), 0, 255), q = clamp(round(v*inv) + z, 0, 255),
                            v^ = (q - z)*step; the offset[] slot of the group then holds z */
  uint32_t range;        /* QV2_ABSMAX and QV2_MINMAX take the group's observed range (|.| max for
                            the symmetric scheme, [min,max] for the asymmetric one);
                            QV2_PERCENTILE additionally clips it to the tensor's |x| percentile;
                            QV2_PERCENTILE_GROUP clips every group to the percentile of its own
                            |x| histogram (the same as QV2_PERCENTILE for QV2_PER_TENSOR) */
  uint32_t flags;        /* pair mode: QV2_PAIR_REQUANT (default) re-quantizes y on x's grid and
                            measures x - dequant(q(y)); QV2_PAIR_RAW measures x - y.
                            QV2_STORE_CODES writes the 8-bit codes (see qv2_quant_metrics). */
  double percentile;     /* in [0,1], e.g. 0.9999; read only by the two percentile range modes */
} qv2_tensor_desc;

/* Ranking parameters (Algorithm 2, RankLayersBySensitivity; Eq. 16; Eq. 17). */
typedef struct {
  double w_gain;           /* weight of the weight-SQNR delta in the score (the paper gives the
                              weight list "more weight" without a number; 2.0 is the usual choice) */
  double a_gain;           /* weight of the activation-SQNR delta (1.0) */
  double mse_factor;       /* a layer whose MSE exceeds mse_factor x the mean MSE goes to the top
                              of the list; the paper uses 5 */
  double sqnr_cap_db;      /* SQNR values are clamped to +-cap before differencing (200) */
  uint32_t select_mode;    /* QV2_BY_COUNT | QV2_BY_BOPS_RATE */
  uint32_t keep_count;     /* QV2_BY_COUNT: how many list entries stay FP32 */
  uint32_t rate_permyriad; /* QV2_BY_BOPS_RATE: requested BOPs-reduction rate, 0..10000
                              (0 = everything FP32, 10000 = everything int8) */
  uint32_t outlier_order;  /* order among the layers whose MSE exceeds the threshold:
                              QV2_OUTLIERS_BY_SEVERITY (0): most severe first;
                              QV2_OUTLIERS_LITERAL: as Algorithm 2's RankLayersBySensitivity is
                              printed -- it walks the layers in order and puts each outlier at the
                              head of the list as it meets it, so the outliers end in reverse
                              layer order (the last one met stands first) */
} qv2_rank_cfg;

/* Creates a context bound to CUDA device `device` and to `stream` (a cudaStream_t, borrowed, may
 * be NULL for the default stream).  Allocates a small amount of device and pinned host scratch. */
int qv2_create(qv2_ctx** out, int device, void* stream);
int qv2_destroy(qv2_ctx* ctx);
/* Static, human-readable name of a status code. */
const char* qv2_status_string(int status);
/* cudaError_t of the most recent failing CUDA call of this context (0 when none). */
int qv2_last_cuda_error(const qv2_ctx* ctx);
/* Number of kernel launches this context has enqueued since it was created. */
uint64_t qv2_launch_count(const qv2_ctx* ctx);
/* Number of times this context has synchronised its stream on the host (tile-table rebuilds,
 * qv2_check_nonfinite, qv2_sweep_model_host, qv2_sweep_graph_create). */
uint64_t qv2_sync_count(const qv2_ctx* ctx);

/*
 * Order in which the phases visit the tensors.  The paper's calibration stage and the loop of
 * Algorithm 2 pass over each tensor three times (range, histogram, error metrics), each pass
 * needing a result of the one before.
 *   QV2_SCHEDULE_PHASE_MAJOR (default): one launch per phase over the whole model; every pass
 *     reads its tensors from HBM.  Right for tensors far larger than L2.
 *   QV2_SCHEDULE_L2_CHUNKED: consecutive tensors are grouped into stages whose reference tensors
 *     (x) hold at most chunk_bytes together; the phases run stage by stage, so the second and third
 *     pass over a stage find x in L2.  Tensors larger than chunk_bytes gather in stages of their
 *     own.  qv2_calibrate runs range -> histogram per stage; qv2_sweep_model (and its captured
 *     form) runs range -> histogram -> metrics per stage.  Results are the same bits for integer
 *     outputs and parameters; sums are added in a stage-dependent order (same tolerances).  Plans
 *     with QV2_PERCENTILE_GROUP tensors keep one stage.
 *   QV2_SCHEDULE_AUTO: whichever measured faster for the plan's sizes.  On a B200 that is
 *     phase-major for every size tried (62 MB to 15 GB per pass): L2 serves a re-read at about
 *     2.2 times the HBM rate and only for stages up to ~32 MB, which does not pay for the
 *     additional launches, so AUTO currently never chunks.
 * chunk_bytes: 0 selects the default (48 MiB, well under half of a B200's 126 MB L2).
 * Takes effect with the next call; QV2_ERR_UNSUPPORTED while a captured pass of this context lives.
 */
int qv2_set_schedule(qv2_ctx* ctx, uint32_t schedule, uint64_t chunk_bytes);
/*
 * Where a tensor's partial results (per-block ranges, histogram counts, partial sums) are folded
 * into its outputs.  QV2_FOLD_SEPARATE: by a small kernel after each streaming kernel (one block
 * per tensor); the streaming kernels then carry no fold code, no fences and no per-tensor
 * barriers.  QV2_FOLD_FUSED: inside the streaming kernel, by the block that finishes the tensor
 * last (found with an atomic ticket; nobody waits) -- one launch per phase instead of two, paid
 * for with a barrier per tensor and block.  QV2_FOLD_AUTO (default) currently always takes the
 * separate form, which measured faster on every workload from 62 MB to 15 GB; the fused form is
 * kept for callers to whom the number of launches matters more.  The outputs do not depend on
 * the choice.  QV2_ERR_UNSUPPORTED while a captured pass of this context lives.
 */
int qv2_set_fold_mode(qv2_ctx* ctx, uint32_t mode);
/*
 * How the kernels of a pass follow one another on the stream.  On (default): every kernel is
 * launched as a programmatic dependent of the one before it, so its launch latency and its
 * prologue overlap the tail of its predecessor; each kernel waits (in hardware, at its first
 * instruction that touches memory) until the predecessor has completed and its writes are
 * visible, so results are the same as with ordinary launches.  Off: ordinary stream order.
 * The first kernel of a call treats whatever precedes it on the stream the same way, which is safe
 * for any predecessor.  QV2_ERR_UNSUPPORTED while a captured pass of this context lives.
 */
int qv2_set_dependent_launch(qv2_ctx* ctx, int on);
/*
 * Measurement aid (no counterpart in the paper): with timing on, qv2_calibrate on a single-stage
 * plan records CUDA events on the context's stream before its range phase, between the range
 * phase and the histogram phase, and after the histogram phase (per-group histograms included).
 * qv2_calibrate_phase_ms waits for the last of them (a host synchronisation, counted by
 * qv2_sync_count) and returns the two durations of the most recent qv2_calibrate call in
 * milliseconds.  QV2_ERR_UNSUPPORTED when timing is off, when no timed call has been made, or when
 * the last call ran a multi-stage plan or inside a stream capture (no events are recorded then).
 * The results of qv2_calibrate are the same either way.
 */
int qv2_set_phase_timing(qv2_ctx* ctx, int on);
int qv2_calibrate_phase_ms(qv2_ctx* ctx, float* range_ms, float* hist_ms);
/* Number of stages of the context's current plan (1 for phase-major; 0 before the first call). */
uint32_t qv2_stage_count(const qv2_ctx* ctx);
/* Sum over descs of the number of quantization groups (1 or `channels`).  Host only. */
uint64_t qv2_group_count(const qv2_tensor_desc* descs, uint32_t n);

/*
 * Convolution + batch-normalisation folding, Eq. 10-12: the pre-pass that produces the weights of
 * the fused graph, on which the mixed-precision decision is applied.  Per output channel c:
 *   s_c = gamma_c / sqrt(var_c);  w_out[c][k] = s_c * w[c][k];  bias_out[c] = s_c*(bias_c - mean_c) + beta_c
 * each operation rounded once in binary32, in that order.  As printed in the paper there is no
 * epsilon under the root: the caller adds it to var if its framework uses one; var_c <= 0 gives
 * Inf/NaN in that channel.
 * w, w_out: device, [channels][inner] fp32; w_out may be w itself (folding in place), but must not
 * overlap it otherwise.  bias: device [channels] or NULL
 * (zeros).  gamma, beta, mean, var: device [channels].  bias_out: device [channels] or NULL.
 */
int qv2_fold_batchnorm(qv2_ctx* ctx, const float* w, const float* bias, const float* gamma,
                       const float* beta, const float* mean, const float* var,
                       uint64_t channels, uint64_t inner, float* w_out, float* bias_out);

/*
 * Calibration: step 1 of the paper's method overview (range statistics of every layer's weights
 * and activations) together with its calibration stage (a histogram of each layer's value range),
 * followed by the scale computation of step 2 (Eq. 4 for symmetric weights, Eq. 2 for the affine
 * form).
 *
 * For every group g of every tensor: gmin/gmax = min/max over the group's finite elements,
 * gabsmax = max(|gmin|,|gmax|) (a zero is returned as +0).  For every tensor t whose range is
 * QV2_PERCENTILE: hist[t*2048 + j] counts the elements with min(2047, trunc(|x| * fl(2048/A))) == j,
 * A the tensor's absmax, and clip[t] is the upper edge of the bin in which the cumulative count
 * first reaches ceil(percentile * N); for the other tensors clip[t] = A and their histogram rows
 * are zero.  Quantization parameters per group, all in binary32 with one rounding per operation:
 *   QV2_SYM_I8:  R = absmax_g (min(absmax_g, clip) under QV2_PERCENTILE);
 *                step = R/127, inv = 127/R, offset = 0
 *   QV2_ASYM_U8: lo = min_g, hi = max_g (clipped to [-clip, clip] under QV2_PERCENTILE);
 *                step = (hi-lo)/255, inv = 255/(hi-lo), offset = lo
 * A degenerate range gives step = inv = 1.
 *
 * descs: host array of n descriptors (x device pointers; y is not read here).
 * gmin, gmax, gabsmax, step, inv, offset: device, qv2_group_count(descs,n) floats each, required.
 * hist: device, n*2048 uint64, or NULL when the histograms are not wanted (they are then kept in
 *       context scratch).  clip: device, n floats, required.  nonfinite: device, n uint64, required.
 * Limits: 1 <= n <= 65535; channels and the total group count < 2^32.
 * Errors: QV2_ERR_NULL, _ARG, _ALIGN, _SIZE, _NOMEM, _CUDA.  On an argument error nothing has
 * been launched.
 */
int qv2_calibrate(qv2_ctx* ctx, const qv2_tensor_desc* descs, uint32_t n,
                  float* gmin, float* gmax, float* gabsmax,
                  uint64_t* hist, float* clip,
                  float* step, float* inv, float* offset,
                  uint64_t* nonfinite);

/*
 * qv2_calibrate with the per-channel form of the percentile clip (range QV2_PERCENTILE_GROUP on a
 * QV2_PER_CHANNEL tensor).  The paper's calibration keeps one histogram per layer; a per-channel
 * quantizer whose channels differ in scale by orders of magnitude gets nothing from a clip taken
 * over the whole tensor, so this mode repeats the construction per group: group g gets its own
 * 2048-bin histogram of |x| on [0, absmax_g], bin = min(2047, trunc(|x| * fl(2048/absmax_g))), and
 * its own clip_g (same cumulative-count rule as clip[t]); its parameters are those of
 * QV2_PERCENTILE with clip_g in place of the tensor's clip.  For such a tensor clip[t] is the
 * tensor's absmax and its row of hist stays zero.  Both calls accept the mode; this one can also
 * return the per-group data:
 * group_hist: device or NULL (context scratch): one 2048-entry uint64 histogram per group of every
 *   QV2_PERCENTILE_GROUP per-channel tensor, those tensors in descriptor order, their groups in
 *   channel order; qv2_group_hist_count gives the number of histograms.
 * group_clip: device or NULL: qv2_group_count floats, the clip bound applied to each group
 *   (clip_g in this mode, the tensor's clip[t] otherwise).
 */
int qv2_calibrate_ex(qv2_ctx* ctx, const qv2_tensor_desc* descs, uint32_t n,
                     float* gmin, float* gmax, float* gabsmax,
                     uint64_t* hist, float* clip,
                     float* step, float* inv, float* offset,
                     uint64_t* nonfinite, uint64_t* group_hist, float* group_clip);
/* Number of per-group histograms qv2_calibrate_ex keeps for these descriptors.  Host only. */
uint64_t qv2_group_hist_count(const qv2_tensor_desc* descs, uint32_t n);

/*
 * Turns the device-side non-finite counters of qv2_calibrate into a status: synchronises the
 * context's stream, reads nonfinite[0..n) (device) and returns QV2_ERR_NONFINITE if any tensor
 * held a NaN or Inf (first_bad, host, nullable, receives the index of the first such tensor),
 * else QV2_OK.  The other calls never synchronise for this; data errors are reported only here
 * and by qv2_sweep_model_host.
 */
int qv2_check_nonfinite(qv2_ctx* ctx, const uint64_t* nonfinite, uint32_t n, uint32_t* first_bad);

/*
 * Fused fake-quantize + error reduction: step 3 of the method overview (per-layer SQNR and MSE
 * between the original and the quantized model's weights and activations), i.e. CalculateSQNR /
 * CalculateMSE of Algorithm 2 over every element, with the quantizer of Eq. 1 / Eq. 5 and the
 * dequantizer of Eq. 3; SQNR is Eq. 6 and MSE is Eq. 7.
 *
 * Per element of the tensor v being quantized (x in self mode, y in QV2_PAIR_REQUANT):
 *   t = fl(fl(v - offset_g) * inv_g);  q = clamp(round_half_even(t), qmin, qmax);
 *   v^ = q*step_g + offset_g;          e = x - v^          (QV2_PAIR_RAW: e = x - y, no codes)
 * Per tensor: sse = sum e^2, sig = sum x^2 (the signal is always the reference tensor x),
 * mse = sse/N, sqnr_db = 10 log10(sig/sse) (+inf when sse == 0, -inf when sig == 0 < sse).
 * Squares are accumulated in binary32 within a tile (chains of 16 additions), then in binary64 in
 * a fixed order, so two runs on the same GPU model give identical bits.  Because the first level
 * is binary32, tensors whose x^2 or e^2 leave its range (|x| beyond roughly 1e-18 .. 1e18) lose
 * accuracy.
 *
 * descs: host, n descriptors (x and, for pair mode, y device pointers).
 * step, inv, offset: device, per-group parameters in qv2_calibrate's layout.
 * codes: NULL, or a host array of n device pointers; for a tensor with QV2_STORE_CODES set and a
 *        non-NULL entry, one byte per element is written (int8 for QV2_SYM_I8, uint8 otherwise).
 * sse, sig, mse, sqnr_db: device, n doubles each, required.
 * Errors: as qv2_calibrate, plus QV2_ERR_ARG for QV2_PAIR_RAW without y.
 */
int qv2_quant_metrics(qv2_ctx* ctx, const qv2_tensor_desc* descs, uint32_t n,
                      const float* step, const float* inv, const float* offset,
                      void* const* codes,
                      double* sse, double* sig, double* mse, double* sqnr_db);

/*
 * qv2_quant_metrics with one more local metric: the cosine similarity of Eq. 8, one of the
 * metrics the paper evaluates beside SQNR and MSE (and then sets aside).  cosine[t] =
 * A.B / (|A| |B|) with A the reference tensor x and B the tensor it is compared with: the
 * dequantized copy of x (self mode), the dequantized re-quantization of y (QV2_PAIR_REQUANT) or y
 * itself (QV2_PAIR_RAW).  It costs one more fused multiply-add per element: with e = A - B,
 * A.B = sig - sum(x e) and |B|^2 = sig - 2 sum(x e) + sse.  A zero vector gives 0.  Accuracy:
 * 1e-7 absolute in general; when B is a quantized copy of A (cos within 1e-2 of 1) the distance
 * 1 - cos is good to 1e-4 relative.
 * cosine: device, n doubles, or NULL (then this is exactly qv2_quant_metrics).
 */
int qv2_quant_metrics_ex(qv2_ctx* ctx, const qv2_tensor_desc* descs, uint32_t n,
                         const float* step, const float* inv, const float* offset,
                         void* const* codes,
                         double* sse, double* sig, double* mse, double* sqnr_db, double* cosine);

/*
 * KL divergence (Eq. 9), the fourth local metric the paper considers (and sets aside):
 * kl[t] = sum_j P_j ln(P_j / Q_j) in nats, P the distribution of the reference tensor x and Q that
 * of the tensor it is compared with (dequantized x, dequantized re-quantized y, or y under
 * QV2_PAIR_RAW).  The paper gives no discretisation; here both are binned on the same
 * QV2_KL_BINS = 128 linear bins of |value| over [0, A], A the tensor-wide absmax of x
 * (bin = min(127, trunc(|v| * fl(128/A))), values beyond A in the last bin), with add-one
 * smoothing: P_j = (count_j + 1) / (N + 128).  The compared value is formed in binary32 as
 * fl(fl(q*step) + offset) (fl((q - z)*step) with a zero point).  Non-finite values are skipped.
 * This is a separate pass over the tensors (4 or 8 bytes per element) and not part of qv2_sweep_model.
 *
 * step, inv, offset, gabsmax: device, per group, as produced by qv2_calibrate.
 * kl: device, n doubles.  hists: device, n*2*128 uint64 (per tensor the histogram of x, then that
 * of the compared tensor), or NULL (kept in context scratch).
 */
#define QV2_KL_BINS 128
int qv2_kl_divergence(qv2_ctx* ctx, const qv2_tensor_desc* descs, uint32_t n,
                      const float* step, const float* inv, const float* offset, const float* gabsmax,
                      double* kl, uint64_t* hists);

/*
 * Sensitivity list and mixed-precision layer set: step 4 of the overview, "CalculateSQNRdeltas",
 * "CalculateAverage" and "RankLayersBySensitivity" of Algorithm 2, the SQNR delta of Eq. 16 and
 * the BOPs-reduction rate of Eq. 17 (normalised so that a fully quantized model is 100 %).
 *
 *   delta_0 = 0, delta_n = (sqnr[n]-sqnr[n-1]) / (pos[n]-pos[n-1]) after clamping sqnr to +-cap;
 *   score_n = w_gain*delta_w_n + a_gain*delta_a_n;
 *   severity_n = max(mse_w[n]/mean(mse_w), mse_a[n]/mean(mse_a)) (a zero mean contributes 0);
 *   order = layers with severity > mse_factor, most severe first (or in reverse layer order, see
 *           qv2_rank_cfg.outlier_order), then the others by ascending score; ties keep layer
 *           order.  A NaN score sorts last, a NaN severity counts as 0.
 *   QV2_BY_COUNT keeps order[0..keep_count) in FP32; QV2_BY_BOPS_RATE keeps the longest prefix for
 *   which (MACs of the still-quantized layers)/(all MACs) >= rate_permyriad/10000.
 *
 * sqnr_w, mse_w, sqnr_a, mse_a: device, n_layers doubles.  macs: device, n_layers uint64, or NULL
 * (every layer counts 1).  pos: device, n_layers doubles, or NULL (positions 0,1,2,...).
 * cfg: host.  order: device uint32[n_layers]; keep_fp32: device uint8[n_layers]; n_keep: device uint32.
 * Limits: 1 <= n_layers <= 8192 (QV2_ERR_SIZE).  Results are bit-exact functions of the inputs.
 */
int qv2_rank_layers(qv2_ctx* ctx, uint32_t n_layers,
                    const double* sqnr_w, const double* mse_w,
                    const double* sqnr_a, const double* mse_a,
                    const uint64_t* macs, const double* pos,
                    const qv2_rank_cfg* cfg,
                    uint32_t* order, uint8_t* keep_fp32, uint32_t* n_keep);

/*
 * qv2_rank_layers with fusion groups.  The paper notes that fusion-capable operators (convolution,
 * batch normalisation, add, ReLU) may have their places in the list adjusted so that they can be
 * fused and share one bit-width, without saying how; this library's reading: fuse_group[i] is the
 * id of layer i's fusion group or QV2_NO_GROUP.  The list of qv2_rank_layers is walked from the
 * top; where the first member of a group stands, the whole group is placed in layer order, and
 * its other members leave their old places.  The FP32-kept prefix never splits a group: by count
 * it is the longest run of whole groups with at most keep_count layers, by rate it grows group
 * by group while the rate still holds.
 * fuse_group: device, n_layers uint32, or NULL (then this is exactly qv2_rank_layers).
 */
#define QV2_NO_GROUP 0xFFFFFFFFu
int qv2_rank_layers_ex(qv2_ctx* ctx, uint32_t n_layers,
                       const double* sqnr_w, const double* mse_w,
                       const double* sqnr_a, const double* mse_a,
                       const uint64_t* macs, const double* pos, const uint32_t* fuse_group,
                       const qv2_rank_cfg* cfg,
                       uint32_t* order, uint8_t* keep_fp32, uint32_t* n_keep);

/* Device buffers of one full-model pass; every pointer is device memory owned by the caller. */
typedef struct {
  float *gmin, *gmax, *gabsmax, *step, *inv, *offset;   /* qv2_group_count floats each */
  uint64_t* hist;                                       /* n_tensors*2048, or NULL */
  float* clip;                                          /* n_tensors */
  uint64_t* nonfinite;                                  /* n_tensors */
  double *sse, *sig, *mse, *sqnr_db;                    /* n_tensors each */
  uint32_t* order;                                      /* n_layers */
  uint8_t* keep_fp32;                                   /* n_layers */
  uint32_t* n_keep;                                     /* 1 */
} qv2_sweep_buffers;

/*
 * One full sensitivity pass over a model (Algorithm 2 end to end): qv2_calibrate, qv2_quant_metrics
 * and qv2_rank_layers chained on the context's stream.  Layout of descs: descs[l] is the weight
 * tensor of layer l and descs[n_layers + l] its activation tensor (l < n_layers); descriptors
 * beyond 2*n_layers are calibrated and measured but do not enter the ranking.
 * macs, pos: device or NULL as in qv2_rank_layers.  Requires n_tensors >= 2*n_layers.
 */
int qv2_sweep_model(qv2_ctx* ctx, const qv2_tensor_desc* descs, uint32_t n_tensors,
                    uint32_t n_layers, const uint64_t* macs, const double* pos,
                    const qv2_rank_cfg* cfg, const qv2_sweep_buffers* bufs);

/*
 * The pass of qv2_sweep_model captured once in a CUDA graph and replayed with a single launch.
 * Algorithm 2 on a small model is a chain of short kernels whose launch overhead exceeds their
 * run time; replaying a captured chain removes it (SqueezeNet shapes: about 50 us -> 23 us per pass).
 * qv2_sweep_graph_create runs one ordinary pass first (argument checks, tile tables, scratch
 * sizing -- results are written as usual), then captures an identical pass on the context's stream;
 * it needs a context created on a non-default stream (QV2_ERR_UNSUPPORTED otherwise) and
 * synchronises that stream.  The graph reads the same tensor and buffer ADDRESSES on every
 * replay: refill the tensors in place, do not move or free them while the graph lives, and do not
 * destroy the context before the graph.  It also holds the addresses of the context's tile tables
 * and scratch: while a graph of a context lives, every other call on that context must use the
 * descriptor set the graph was captured with (calls with another set, or that would have to move
 * scratch, return QV2_ERR_UNSUPPORTED and leave the graph intact); use a second context for other
 * models.  qv2_sweep_graph_launch enqueues one replay on the context's stream and returns.
 */
typedef struct qv2_graph qv2_graph;
int qv2_sweep_graph_create(qv2_ctx* ctx, const qv2_tensor_desc* descs, uint32_t n_tensors,
                           uint32_t n_layers, const uint64_t* macs, const double* pos,
                           const qv2_rank_cfg* cfg, const qv2_sweep_buffers* bufs, qv2_graph** out);
int qv2_sweep_graph_launch(qv2_graph* graph);
int qv2_sweep_graph_destroy(qv2_graph* graph);

/* Host-side results of qv2_sweep_model_host; every pointer is host memory owned by the caller. */
typedef struct {
  double *mse, *sqnr_db;       /* n_tensors each */
  uint64_t* nonfinite;         /* n_tensors */
  uint32_t* order;             /* n_layers */
  uint8_t* keep_fp32;          /* n_layers */
  uint32_t* n_keep;            /* 1 */
} qv2_host_results;

/*
 * The same pass for tensors that live in HOST memory (pinned memory makes the copies fast):
 * every x / y of descs is a host pointer; the call copies them into `staging` (device, caller
 * owned, at least qv2_staging_bytes(descs, n_tensors, n_layers) bytes), runs qv2_sweep_model on
 * the copies, copies the results back into `out`, and synchronises the stream before returning.
 * macs, pos: HOST arrays or NULL.  Returns QV2_ERR_NONFINITE (results still written) when any
 * input element was NaN or Inf.  QV2_STORE_CODES is not available through this call.
 */
int qv2_sweep_model_host(qv2_ctx* ctx, const qv2_tensor_desc* descs, uint32_t n_tensors,
                         uint32_t n_layers, const uint64_t* macs, const double* pos,
                         const qv2_rank_cfg* cfg, void* staging, uint64_t staging_bytes,
                         const qv2_sweep_buffers* bufs, const qv2_host_results* out);
uint64_t qv2_staging_bytes(const qv2_tensor_desc* descs, uint32_t n_tensors, uint32_t n_layers);

/*
 * The fake-quantize + error reduction of qv2_quant_metrics for ONE tensor, for callers that must
 * not allocate.  (The paper has no counterpart to this call; it exists for the library's users.)
 *
 * Who needs it: code that runs where cudaMalloc / cudaFree are off limits -- inside a region whose
 * memory footprint was fixed up front (a serving process that has handed all device memory to its
 * own pool), in a latency-critical loop where an allocation would stall the device, or in a host
 * callback.  The regular entry points keep tile tables and partial sums in context scratch that
 * grows with cudaMalloc; this one takes no context and calls no allocator of any kind.  Instead
 * its partial sums (one pair of doubles per warp and per 16384-element tile) live in a fixed
 * 1 MiB array that is part of the library image: every GPU that loads the library holds that
 * 1 MiB until the process ends, whether or not this call is ever used.
 *
 * desc: host, one descriptor (x and, for pair mode, y are device pointers; QV2_STORE_CODES is not
 * accepted).  step, inv, offset: device, this tensor's per-group parameters (group 0 first), e.g.
 * a slice of qv2_calibrate's output.  result4: device, 4 doubles {sse, sig, mse, sqnr_db}, defined
 * as in qv2_quant_metrics.  stream: cudaStream_t or NULL.  The work is enqueued and the call
 * returns; results are valid once the stream has been synchronised.
 *
 * Limit: outer*channels*inner <= QV2_NOALLOC_MAX_ELEMS, and no more than
 * QV2_NOALLOC_MAX_ELEMS/16384 tiles (per-channel rows of 4096 elements or more are cut at row
 * boundaries, so very ragged shapes reach the tile limit earlier).  Larger tensors are refused
 * with QV2_ERR_SIZE before anything is launched; split them or use qv2_quant_metrics.
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress) and the
 * SM count; make that first call outside any stream capture.  All calls on a device share the one
 * array, which still holds the previous call's partial sums: each call overwrites every slot it
 * later reads, so nothing has to be cleared, but two calls that overlap on the GPU (different
 * streams, or host threads racing) corrupt each other -- serialise them.  Sums are added in a
 * different order than in qv2_quant_metrics, so the two agree to rounding (the same tolerances:
 * 1e-5 relative on MSE, 1e-3 dB on SQNR), not bit for bit.
 * Errors: QV2_ERR_NULL, _ARG, _ALIGN, _SIZE, _CUDA.
 */
#define QV2_NOALLOC_MAX_ELEMS (134217728ull) /* 2^27 elements = 8192 tiles -> 65536 slots = 1 MiB */
int qv2_quant_metrics_noalloc(int device, void* stream, const qv2_tensor_desc* desc,
                              const float* step, const float* inv, const float* offset,
                              double* result4);

/*
 * Host-only view of the work decomposition, for tests: cuts the tensors into the tiles the
 * kernels walk (no GPU needed, tensor pointers are not dereferenced).  Each tile is reported as
 * 4 uint64: {tensor, first element, element count, kind (0 = one group per tile, 1 = whole rows)}.
 * Returns the number of tiles, or a negative status; at most max_tiles are written.
 */
int64_t qv2_debug_plan_tiles(const qv2_tensor_desc* descs, uint32_t n, uint64_t* out, uint64_t max_tiles);

#ifdef __cplusplus
}
#endif
#endif /* QV2_H_ */
