// |x| histogram for percentile clipping (the paper's calibration stage keeps a histogram of each
// layer's value range): 2048 linear bins on [0, absmax] per tensor, counted exactly.
//
// Each CTA keeps a private 2048 x u32 histogram in shared memory across all the tiles it walks of
// one tensor and merges it into the tensor's 64-bit accumulation histogram only when it moves to
// another tensor; the CTA that merges last turns the counts into the clip and the quantization
// parameters.  Counts are integers, so the result does not depend on the order of the atomics.
#include "qv2_device.cuh"

namespace qv2 {

namespace {

// bin = min(2047, trunc(fl(|v| * w))).  For 0 <= f < 2^23, adding 2^23 with round-toward-zero
// leaves trunc(f) in the low mantissa bits; larger or NaN f give a large index that the min
// clamps, so the shared-memory index is always in range.
__device__ __forceinline__ uint32_t bin_of(float v, float w) {
  const float f = __fmul_rn(fabsf(v), w);
  const uint32_t b = __float_as_uint(__fadd_rz(f, 8388608.0f)) - 0x4B000000u;
  return min(b, (uint32_t)(kBins - 1));
}

// Bin 0 is counted in a register instead of shared memory: half of a post-ReLU tensor sits there,
// and it would otherwise be many lanes of a warp adding to one shared-memory word.  (Doing the
// same for the top bin, where ReLU6-saturated elements sit, was measured and cost 1.2-1.5 % of the
// pass on every workload, MobileNet-v2 shapes included: the kernel is bound by instruction issue,
// and the second test costs more than the conflicts it avoids.)
struct EdgeCount {
  uint32_t lo;
};
template <bool CAREFUL>
__device__ __forceinline__ void hist_elem(float v, float w, uint32_t* sh, EdgeCount& edge) {
  if (CAREFUL && !isfinite(v)) return;
  const uint32_t b = bin_of(v, w);
  if (b == 0) ++edge.lo;
  else atomicAdd(sh + b, 1u);
}
__device__ __forceinline__ void flush_edges(uint32_t* sh, EdgeCount& edge) {
  if (edge.lo) atomicAdd(sh, edge.lo);
  edge.lo = 0;
}

template <bool CAREFUL, class T>
__device__ __forceinline__ void hist_flat(const T* __restrict__ x, uint32_t count, float w,
                                          uint32_t* sh, EdgeCount& zeros) {
  const FlatSplit s = split_flat(x, count);
  const T* xv = x + s.head;
  constexpr uint32_t U = 4;
  uint32_t j = threadIdx.x;
  const uint32_t n_full = s.nvec / (U * kThreads) * (U * kThreads);   // rounds in which every thread has U groups
  for (; j < n_full; j += U * kThreads) {
    float4 v[U];
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) v[u] = ld_vec_at(xv, j + u * kThreads);
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) {
      hist_elem<CAREFUL>(v[u].x, w, sh, zeros); hist_elem<CAREFUL>(v[u].y, w, sh, zeros);
      hist_elem<CAREFUL>(v[u].z, w, sh, zeros); hist_elem<CAREFUL>(v[u].w, w, sh, zeros);
    }
  }
  if (n_full < s.nvec) {            // what is left: one predicated round
    float4 v[U];
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) v[u] = ld_vec_at(xv, min(j + u * kThreads, s.nvec - 1u));   // in bounds, maybe unused
#pragma unroll
    for (uint32_t u = 0; u < U; ++u)
      if (j + u * kThreads < s.nvec) {
        hist_elem<CAREFUL>(v[u].x, w, sh, zeros); hist_elem<CAREFUL>(v[u].y, w, sh, zeros);
        hist_elem<CAREFUL>(v[u].z, w, sh, zeros); hist_elem<CAREFUL>(v[u].w, w, sh, zeros);
      }
  }
  if (threadIdx.x < s.head) hist_elem<CAREFUL>(Ld<T>::one(x + threadIdx.x), w, sh, zeros);
  if (threadIdx.x < s.tail)
    hist_elem<CAREFUL>(Ld<T>::one(x + s.head + 4u * s.nvec + threadIdx.x), w, sh, zeros);
}

template <class T>
__device__ __forceinline__ void hist_tile(const T* x, uint32_t count, float w, bool careful, uint32_t* sh,
                                          EdgeCount& zeros) {
  if (careful) hist_flat<true>(x, count, w, sh, zeros);
  else hist_flat<false>(x, count, w, sh, zeros);
}

// Folds the histogram of one tensor once every CTA that owns a tile of it has merged its counts:
// percentile clip, then the quantization parameters of the tensor's groups.
// T = clamp(ceil(p * Nf), 1, Nf) with Nf the histogram total; k* = first bin whose cumulative
// count reaches T; clip = upper edge of bin k* (absmax itself for the last bin).  The counts are
// copied to the caller's histogram (when it wants one) and the accumulation row is put back to
// zero for the next pass.  Runs in the CTA that drew the tensor's last ticket; the counts, written
// by other CTAs, are read through L2.
__device__ __noinline__ void clip_fold_tensor(const CalibArgs& a, uint32_t t) {
  __shared__ unsigned long long scan[kThreads];
  __shared__ uint32_t kstar_s;
  const uint32_t tid = threadIdx.x;
  const TensorRec tr = a.tensors[t];
  const float A = a.tensor_absmax[t];
  constexpr uint32_t kPer = kBins / kThreads;
  unsigned long long* acc = a.hist_acc + (size_t)tr.hist_index * kBins;
  unsigned long long local[kPer], mine = 0;
#pragma unroll
  for (uint32_t i = 0; i < kPer; ++i) {
    local[i] = __ldcg(acc + tid * kPer + i);
    acc[tid * kPer + i] = 0ull;
    mine += local[i];
  }
  if (a.hist) {
#pragma unroll
    for (uint32_t i = 0; i < kPer; ++i) a.hist[(size_t)t * kBins + tid * kPer + i] = local[i];
  }
  scan[tid] = mine;
  if (tid == 0) { kstar_s = kBins - 1; a.hist_tickets[t] = 0u; }
  __syncthreads();
  for (uint32_t o = 1; o < kThreads; o <<= 1) {
    const unsigned long long add = tid >= o ? scan[tid - o] : 0ull;
    __syncthreads();
    scan[tid] += add;
    __syncthreads();
  }
  const unsigned long long nf = scan[kThreads - 1], excl = scan[tid] - mine;
  float c = A;
  if (nf != 0ull) {
    const double tt = ceil(__dmul_rn(tr.percentile, (double)nf));
    unsigned long long T;
    if (!(tt >= 1.0)) T = 1ull;
    else if (tt >= (double)nf) T = nf;
    else T = (unsigned long long)tt;
    if (excl < T && T <= excl + mine) {      // exactly one thread owns the target count
      unsigned long long cum = excl;
#pragma unroll
      for (uint32_t i = 0; i < kPer; ++i) {
        cum += local[i];
        if (cum >= T) { kstar_s = tid * kPer + i; break; }
      }
    }
    __syncthreads();
    const uint32_t k = kstar_s;
    if (k != kBins - 1) c = __fmul_rn((float)(k + 1), __fdiv_rn(A, (float)kBins));
  }
  if (tid == 0) a.clip[t] = c;
  for (uint32_t g = tid; g < tr.n_groups; g += kThreads) {
    const uint32_t G = tr.group_base + g;
    make_qparams(tr.asym, top_code(tr.asym != 0, tr.bits), true, c, a.gmin[G], a.gmax[G], a.gabsmax[G],
                 a.step + G, a.inv + G, a.offset + G);
  }
  __syncthreads();                           // the shared arrays may be reused by the next fold
}

// ANY16 = false: every tensor is binary32, no element-type dispatch.  FOLD as in range_kernel:
// true folds in the CTA that merges a tensor last, false leaves it to clip_fold_kernel.
template <bool ANY16, bool FOLD>
__global__ void __launch_bounds__(kThreads, 4)
hist_kernel(const __grid_constant__ CalibArgs a, const TensorRec* __restrict__ tensors,
            const Tile* __restrict__ tiles, uint32_t n_tiles, uint32_t scan_begin, uint32_t scan_end) {
  __shared__ uint32_t sh[kBins];
  __shared__ uint32_t s_last;
  for (uint32_t b = threadIdx.x; b < kBins; b += kThreads) sh[b] = 0;
  __syncthreads();
  dependency_wait();
  // percentile tensors without elements are owned by no CTA: CTA 0 folds them
  if (FOLD && blockIdx.x == 0)
    for (uint32_t t = scan_begin; t < scan_end; ++t)
      if (tensors[t].range_mode == QV2_PERCENTILE && tensors[t].hist_ctas == 0) clip_fold_tensor(a, t);

  constexpr uint32_t kNone = 0xffffffffu;
  uint32_t cur = kNone, since_flush = 0;
  EdgeCount zeros = {0u};
  uint32_t owed = kNone, drawn = 0;   // FOLD: the tensor before cur and the ticket thread 0 drew for it
  float w = 0.0f;
  bool careful = false;
  // Ticket protocol of the fused fold: after a tensor's merge (and a barrier), thread 0 fences and
  // draws the tensor's ticket without looking at the result; the CTA looks at it at its next
  // tensor boundary and folds the tensor if the ticket was the last one.  The atomic's round
  // trip hides behind the next tensor's stream; nobody waits for another CTA.
  auto settle = [&](uint32_t t) {
    if (threadIdx.x == 0) {
      const bool last = drawn == tensors[t].hist_ctas - 1u;
      if (last) __threadfence();
      s_last = last;
    }
    __syncthreads();
    if (s_last) clip_fold_tensor(a, t);
  };
  for (uint32_t ti = blockIdx.x;; ti += gridDim.x) {
    const bool more = ti < n_tiles;
    Tile tl;
    if (more) tl = load_tile(tiles, ti);
    // merge into the accumulation histogram when the tensor changes, at the end, and before a
    // 32-bit count could overflow (2^14 tiles of 2^14 elements)
    const bool leaving = cur != kNone && (!more || tl.tensor != cur);
    if (leaving || (cur != kNone && since_flush >= 16384u)) {
      flush_edges(sh, zeros);
      __syncthreads();
      unsigned long long* h = a.hist_acc + (size_t)tensors[cur].hist_index * kBins;
      for (uint32_t b = threadIdx.x; b < kBins; b += kThreads) {
        const uint32_t c = sh[b];
        if (c) { atomicAdd(h + b, (unsigned long long)c); sh[b] = 0; }
      }
      __syncthreads();
      since_flush = 0;
      if (FOLD && leaving) {
        if (owed != kNone) settle(owed);
        if (threadIdx.x == 0) { __threadfence(); drawn = atomicAdd(a.hist_tickets + cur, 1u); }
        owed = cur;
      }
    }
    if (!more) {
      allow_dependents();          // this CTA is done: the next kernel may start to launch
      if (FOLD && owed != kNone) settle(owed);
      break;
    }
    if (tl.tensor != cur) {
      cur = tl.tensor;
      const float A = a.tensor_absmax[cur];
      w = (A > 0.0f) ? __fdiv_rn((float)kBins, A) : 0.0f;
      if (!isfinite(w)) w = 0.0f;
      careful = a.nonfinite[cur] != 0ull;
    }
    const TensorRec* tr = tensors + cur;
    if (!ANY16 || tr->dtype == kF32) hist_tile(reinterpret_cast<const float*>(tr->x) + tl.begin, tl.count, w, careful, sh, zeros);
    else if (tr->dtype == kF16) hist_tile(reinterpret_cast<const __half*>(tr->x) + tl.begin, tl.count, w, careful, sh, zeros);
    else hist_tile(reinterpret_cast<const __nv_bfloat16*>(tr->x) + tl.begin, tl.count, w, careful, sh, zeros);
    ++since_flush;
  }
}

// One CTA per tensor of the stage: the fold, for stages whose streaming kernel does not fold.
__global__ void __launch_bounds__(kThreads)
clip_fold_kernel(const __grid_constant__ CalibArgs a, uint32_t tensor_begin) {
  allow_dependents();
  dependency_wait();
  const uint32_t t = tensor_begin + blockIdx.x;
  if (a.tensors[t].range_mode == QV2_PERCENTILE) clip_fold_tensor(a, t);
}

// ------------------------------------------------------------------------------------------------
// Per-group histograms (range mode QV2_PERCENTILE_GROUP on per-channel tensors): the same binning,
// on [0, absmax_g] of each group, one 2048-bin histogram per group.
//
// The pass is group-major: a unit is `rows` segments of `count` contiguous elements of ONE group
// (the same channel of consecutive batch items), about 128 K elements.  A CTA counts a whole unit
// into its shared-memory histogram and merges it into the group's global histogram once, at the
// end of the unit.  Very small groups are packed several to a unit and skip the shared histogram.
__device__ __forceinline__ float bin_scale(float A) {
  float w = (A > 0.0f) ? __fdiv_rn((float)kBins, A) : 0.0f;
  return isfinite(w) ? w : 0.0f;
}

// Exact n / d by one multiply-high, for n * d <= 2^32: with m = floor((2^32 - 1) / d) + 1 the
// product m * d exceeds 2^32 by less than d, so the error of n * m / 2^32 stays below 1 / d.
struct FastDiv {
  uint32_t m, d;
};
__device__ __forceinline__ FastDiv fast_div(uint32_t d) {
  FastDiv f;
  f.d = d; f.m = d > 1u ? 0xFFFFFFFFu / d + 1u : 0u;
  return f;
}
__device__ __forceinline__ uint32_t div_by(uint32_t n, const FastDiv& f) { return f.d > 1u ? __umulhi(n, f.m) : n; }

// `rows` segments of `count` elements, segment r at x + r * seg_stride, walked by the whole CTA as
// ONE index space of 16-byte groups: every thread keeps four loads in flight whatever the segment
// length, and a round that straddles segments costs nothing.  Needs every segment to start on a
// four-element boundary and to hold whole groups, and rows * (count / 4)^2 <= 2^32 (FastDiv).
template <bool CAREFUL, class T>
__device__ __forceinline__ void hist_rows_vec(const T* __restrict__ x, uint32_t rows, uint32_t count,
                                              uint64_t seg_stride, float w, uint32_t* sh, EdgeCount& zeros) {
  constexpr uint32_t U = 4;
  const uint32_t nv = count >> 2, total = rows * nv;
  const FastDiv f = fast_div(nv);
  uint32_t j = threadIdx.x;
  const uint32_t n_full = total / (U * kThreads) * (U * kThreads);
  for (; j < n_full; j += U * kThreads) {
    float4 v[U];
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) {
      const uint32_t idx = j + u * kThreads, r = div_by(idx, f);
      v[u] = ld_vec_at(x + r * seg_stride, idx - r * nv);
    }
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) {
      hist_elem<CAREFUL>(v[u].x, w, sh, zeros); hist_elem<CAREFUL>(v[u].y, w, sh, zeros);
      hist_elem<CAREFUL>(v[u].z, w, sh, zeros); hist_elem<CAREFUL>(v[u].w, w, sh, zeros);
    }
  }
  if (n_full < total) {             // what is left: one predicated round
    float4 v[U];
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) {
      const uint32_t idx = min(j + u * kThreads, total - 1u), r = div_by(idx, f);   // in bounds, maybe unused
      v[u] = ld_vec_at(x + r * seg_stride, idx - r * nv);
    }
#pragma unroll
    for (uint32_t u = 0; u < U; ++u)
      if (j + u * kThreads < total) {
        hist_elem<CAREFUL>(v[u].x, w, sh, zeros); hist_elem<CAREFUL>(v[u].y, w, sh, zeros);
        hist_elem<CAREFUL>(v[u].z, w, sh, zeros); hist_elem<CAREFUL>(v[u].w, w, sh, zeros);
      }
  }
}

// The same index space element by element, for short segments that do not line up with 16-byte
// groups (7x7 maps, odd strides): eight scalar loads in flight per thread.  rows * count^2 <= 2^32.
template <bool CAREFUL, class T>
__device__ __noinline__ void hist_rows_scalar(const T* __restrict__ x, uint32_t rows, uint32_t count,
                                                 uint64_t seg_stride, float w, uint32_t* sh, EdgeCount& zeros) {
  constexpr uint32_t U = 8;
  const uint32_t total = rows * count;
  const FastDiv f = fast_div(count);
  for (uint32_t j0 = 0; j0 < total; j0 += U * kThreads) {
    float v[U];
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) {
      const uint32_t idx = min(j0 + threadIdx.x + u * kThreads, total - 1u), r = div_by(idx, f);
      v[u] = Ld<T>::one(x + r * seg_stride + (idx - r * count));
    }
#pragma unroll
    for (uint32_t u = 0; u < U; ++u)
      if (j0 + threadIdx.x + u * kThreads < total) hist_elem<CAREFUL>(v[u], w, sh, zeros);
  }
}

// One segment handled by one warp: 16-byte loads over the aligned body, scalars at the ends.
template <bool CAREFUL, class T>
__device__ __forceinline__ void hist_segment_warp(const T* __restrict__ x, uint32_t count, uint32_t lane,
                                                  float w, uint32_t* sh, EdgeCount& zeros) {
  const FlatSplit s = split_flat(x, count);
  const T* xv = x + s.head;
  uint32_t j = lane;
  const uint32_t n_full = s.nvec / 128u * 128u;      // rounds in which every lane has four groups
  for (; j < n_full; j += 128) {
    float4 v[4];
#pragma unroll
    for (uint32_t u = 0; u < 4; ++u) v[u] = ld_vec_at(xv, j + 32u * u);
#pragma unroll
    for (uint32_t u = 0; u < 4; ++u) {
      hist_elem<CAREFUL>(v[u].x, w, sh, zeros); hist_elem<CAREFUL>(v[u].y, w, sh, zeros);
      hist_elem<CAREFUL>(v[u].z, w, sh, zeros); hist_elem<CAREFUL>(v[u].w, w, sh, zeros);
    }
  }
  if (n_full < s.nvec) {            // what is left: one predicated round
    float4 v[4];
#pragma unroll
    for (uint32_t u = 0; u < 4; ++u) v[u] = ld_vec_at(xv, min(j + 32u * u, s.nvec - 1u));   // in bounds, maybe unused
#pragma unroll
    for (uint32_t u = 0; u < 4; ++u)
      if (j + 32u * u < s.nvec) {
        hist_elem<CAREFUL>(v[u].x, w, sh, zeros); hist_elem<CAREFUL>(v[u].y, w, sh, zeros);
        hist_elem<CAREFUL>(v[u].z, w, sh, zeros); hist_elem<CAREFUL>(v[u].w, w, sh, zeros);
      }
  }
  if (lane < s.head) hist_elem<CAREFUL>(Ld<T>::one(x + lane), w, sh, zeros);
  if (lane < s.tail) hist_elem<CAREFUL>(Ld<T>::one(x + s.head + 4u * s.nvec + lane), w, sh, zeros);
}

constexpr uint32_t kWarpSegmentMax = 4096;     // unaligned segments shorter than this go one per warp ...
constexpr uint32_t kScalarSegmentMax = 256;    // ... and shorter than this element by element

template <bool CAREFUL, class T>
__device__ __forceinline__ void group_hist_unit(const T* x, const Tile& u, uint64_t seg_stride, float w,
                                                uint32_t* sh, EdgeCount& zeros) {
  const uint64_t nv = u.count >> 2;
  const bool lined_up = (((uintptr_t)x / sizeof(T) | seg_stride | u.count) & 3u) == 0;
  if (lined_up && u.rows * nv * nv <= (1ull << 32)) {
    hist_rows_vec<CAREFUL>(x, u.rows, u.count, seg_stride, w, sh, zeros);
  } else if (u.count >= kWarpSegmentMax) {
    for (uint32_t r = 0; r < u.rows; ++r) hist_flat<CAREFUL>(x + r * seg_stride, u.count, w, sh, zeros);
  } else if (u.count >= kScalarSegmentMax) {
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    for (uint32_t r = warp; r < u.rows; r += kWarps) hist_segment_warp<CAREFUL>(x + r * seg_stride, u.count, lane, w, sh, zeros);
  } else {
    hist_rows_scalar<CAREFUL>(x, u.rows, u.count, seg_stride, w, sh, zeros);   // rows * count <= kGroupUnitElems
  }
}

// Groups of at most kMicroGroupMax elements (fully connected activations: one element per batch
// item and channel): a unit is `nc` CONSECUTIVE channels, all batch items.  Clearing and merging
// a 2048-bin shared histogram per group would cost far more than the group's few elements, so
// each element adds straight into its group's global histogram.  `wtab` (the CTA's shared
// histogram, zero on entry and on exit) holds the nc bin scales meanwhile.
template <bool CAREFUL, class T>
__device__ __noinline__ void micro_groups(const T* __restrict__ x, const Tile& u, uint64_t seg_stride,
                                             const float* __restrict__ gabsmax, uint32_t* wtab,
                                             unsigned long long* h) {
  constexpr uint32_t U = 8;
  const uint32_t nc = u.pack, inner = u.count, run = nc * inner, total = u.rows * run;   // total^2 <= 2^32
  for (uint32_t c = threadIdx.x; c < nc; c += kThreads) wtab[c] = __float_as_uint(bin_scale(gabsmax[c]));
  __syncthreads();
  const FastDiv fr = fast_div(run), fi = fast_div(inner);
  for (uint32_t j0 = 0; j0 < total; j0 += U * kThreads) {
    float v[U];
    uint32_t ch[U];
#pragma unroll
    for (uint32_t k = 0; k < U; ++k) {
      const uint32_t idx = min(j0 + threadIdx.x + k * kThreads, total - 1u), o = div_by(idx, fr), e = idx - o * run;
      ch[k] = div_by(e, fi);
      v[k] = Ld<T>::one(x + o * seg_stride + e);
    }
#pragma unroll
    for (uint32_t k = 0; k < U; ++k)
      if (j0 + threadIdx.x + k * kThreads < total && !(CAREFUL && !isfinite(v[k])))
        atomicAdd(h + (size_t)ch[k] * kBins + bin_of(v[k], __uint_as_float(wtab[ch[k]])), 1ull);
  }
  __syncthreads();
  for (uint32_t c = threadIdx.x; c < nc; c += kThreads) wtab[c] = 0u;
  __syncthreads();
}

template <class T>
__device__ __forceinline__ void group_hist_any(const T* x, const Tile& u, const TensorRec* tr, bool careful,
                                               const float* __restrict__ gabsmax, uint32_t* sh, unsigned long long* h) {
  const uint64_t seg_stride = (uint64_t)tr->channels * tr->inner;
  const float* A = gabsmax + tr->group_base + (uint32_t)u.row0;
  if (u.pack) {
    if (careful) micro_groups<true>(x, u, seg_stride, A, sh, h);
    else micro_groups<false>(x, u, seg_stride, A, sh, h);
    return;
  }
  const float w = bin_scale(A[0]);
  EdgeCount zeros = {0u};
  if (careful) group_hist_unit<true>(x, u, seg_stride, w, sh, zeros);
  else group_hist_unit<false>(x, u, seg_stride, w, sh, zeros);
  // merge: a unit holds fewer than 2^32 elements, so the 32-bit counts cannot have wrapped
  flush_edges(sh, zeros);
  __syncthreads();
  for (uint32_t b = threadIdx.x; b < kBins; b += kThreads) {
    const uint32_t c = sh[b];
    if (c) { atomicAdd(h + b, (unsigned long long)c); sh[b] = 0; }
  }
  __syncthreads();
}

template <bool ANY16>
__global__ void __launch_bounds__(kThreads, 5)
group_hist_kernel(const TensorRec* __restrict__ tensors, const Tile* __restrict__ units, uint32_t n_units,
                  const float* __restrict__ gabsmax, const unsigned long long* __restrict__ nonfinite,
                  unsigned long long* ghist) {
  __shared__ uint32_t sh[kBins];
  for (uint32_t b = threadIdx.x; b < kBins; b += kThreads) sh[b] = 0;
  __syncthreads();
  for (uint32_t ui = blockIdx.x; ui < n_units; ui += gridDim.x) {
    const Tile u = load_tile(units, ui);
    const TensorRec* tr = tensors + u.tensor;
    const bool careful = nonfinite[u.tensor] != 0ull;
    unsigned long long* h = ghist + (size_t)(tr->ghist_first + (uint32_t)u.row0) * kBins;
    if (!ANY16 || tr->dtype == kF32) group_hist_any(reinterpret_cast<const float*>(tr->x) + u.begin, u, tr, careful, gabsmax, sh, h);
    else if (tr->dtype == kF16) group_hist_any(reinterpret_cast<const __half*>(tr->x) + u.begin, u, tr, careful, gabsmax, sh, h);
    else group_hist_any(reinterpret_cast<const __nv_bfloat16*>(tr->x) + u.begin, u, tr, careful, gabsmax, sh, h);
  }
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One warp per group histogram: the group's clip by the same cumulative-count rule as
// clip_fold_tensor, then the group's quantization parameters.
//
// The rule asks for k* = first bin whose cumulative count reaches T.  With A(k) = number of
// elements above bin k that is the same as k* = first k with A(k) <= N - T, and for the usual
// percentiles (close to 1) that bin is near the top; so the warp scans the histogram from the top
// down, 32 bins at a time, and stops at the highest bin b whose count-from-b-upwards exceeds
// N - T: k* = b.  Thousands of 16 KB histograms are then read a few hundred bytes each.  N is the
// group's element count when the tensor holds no NaN or Inf; otherwise the histogram is summed.
__global__ void __launch_bounds__(256)
group_clip_finalize_kernel(const TensorRec* __restrict__ tensors, const uint32_t* __restrict__ owner,
                           uint32_t n_hists, const unsigned long long* __restrict__ ghist,
                           const unsigned long long* __restrict__ nonfinite,
                           const float* __restrict__ gmin, const float* __restrict__ gmax,
                           const float* __restrict__ gabsmax, float* group_clip, float* step, float* inv,
                           float* offset) {
  const uint32_t lane = threadIdx.x & 31u;
  const uint32_t hidx = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (hidx >= n_hists) return;
  const uint32_t t = owner[hidx];
  const TensorRec* tr = tensors + t;
  const uint32_t G = tr->group_base + (hidx - tr->ghist_first);
  const unsigned long long* h = ghist + (size_t)hidx * kBins;
  const float A = gabsmax[G];
  unsigned long long nf;
  if (nonfinite[t] == 0ull) {
    nf = tr->n_elems / tr->n_groups;              // every element of the group was counted
  } else {
    nf = 0;
    for (uint32_t i = 0; i < kBins / 32; ++i) nf += h[i * 32 + lane];
    nf = warp_sum_u64(nf);
  }
  float c = A;
  if (nf != 0ull) {
    const double tt = ceil(__dmul_rn(tr->percentile, (double)nf));
    unsigned long long T;
    if (!(tt >= 1.0)) T = 1ull;
    else if (tt >= (double)nf) T = nf;
    else T = (unsigned long long)tt;
    const unsigned long long rem = nf - T;        // elements allowed above bin k*
    unsigned long long carry = 0;                 // count of the bins above the current 32
    uint32_t kstar = 0;
    for (int i = kBins / 32 - 1; i >= 0; --i) {
      unsigned long long sfx = h[i * 32 + lane];  // inclusive suffix sum over the 32 bins, upwards from this lane
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long up = __shfl_down_sync(0xffffffffu, sfx, o);
        if ((int)lane + o < 32) sfx += up;
      }
      const uint32_t over = __ballot_sync(0xffffffffu, carry + sfx > rem);
      if (over) { kstar = (uint32_t)i * 32u + (31u - (uint32_t)__clz(over)); break; }
      carry += __shfl_sync(0xffffffffu, sfx, 0);
    }
    if (kstar != kBins - 1) c = __fmul_rn((float)(kstar + 1), __fdiv_rn(A, (float)kBins));
  }
  if (lane == 0) {
    if (group_clip) group_clip[G] = c;
    make_qparams(tr->asym, top_code(tr->asym != 0, tr->bits), true, c, gmin[G], gmax[G], A, step + G, inv + G, offset + G);
  }
}

// group_clip for the tensors without per-group histograms: the tensor's clip.
__global__ void __launch_bounds__(256)
fill_group_clip_kernel(const TensorRec* __restrict__ tensors, const float* __restrict__ clip, float* group_clip) {
  const TensorRec* tr = tensors + blockIdx.x;
  if (tr->range_mode == QV2_PERCENTILE_GROUP) return;
  const float c = clip[blockIdx.x];
  for (uint32_t g = threadIdx.x; g < tr->n_groups; g += blockDim.x) group_clip[tr->group_base + g] = c;
}

}  // namespace

uint32_t hist_grid_cap(int sm_count, bool fused) {
  int cache = 0;
  const void* k = fused ? (const void*)hist_kernel<false, true> : (const void*)hist_kernel<false, false>;
  return (uint32_t)persistent_grid(k, &cache, sm_count, 0x7fffffffu);
}
uint32_t group_hist_grid_cap(int sm_count) {
  int cache = 0;
  return (uint32_t)persistent_grid((const void*)group_hist_kernel<false>, &cache, sm_count, 0x7fffffffu);
}

cudaError_t launch_group_hist(const Launch& l, uint32_t grid_cap, bool any16, const TensorRec* tensors,
                              const Tile* tiles, uint32_t n_tiles, const float* gabsmax,
                              const unsigned long long* nonfinite, unsigned long long* ghist) {
  if (n_tiles == 0) return cudaSuccess;
  const uint32_t grid = grid_cap < n_tiles ? (grid_cap ? grid_cap : 1u) : n_tiles;
  if (any16) group_hist_kernel<true><<<grid, kThreads, 0, l.stream>>>(tensors, tiles, n_tiles, gabsmax, nonfinite, ghist);
  else group_hist_kernel<false><<<grid, kThreads, 0, l.stream>>>(tensors, tiles, n_tiles, gabsmax, nonfinite, ghist);
  return cudaGetLastError();
}

cudaError_t launch_group_clip_finalize(const Launch& l, const TensorRec* tensors, const uint32_t* owner,
                                       uint32_t n_hists, const unsigned long long* ghist,
                                       const unsigned long long* nonfinite,
                                       const float* gmin, const float* gmax, const float* gabsmax,
                                       float* group_clip, float* step, float* inv, float* offset) {
  if (n_hists == 0) return cudaSuccess;
  group_clip_finalize_kernel<<<(n_hists + 7) / 8, 256, 0, l.stream>>>(tensors, owner, n_hists, ghist, nonfinite, gmin,
                                                                     gmax, gabsmax, group_clip, step, inv, offset);
  return cudaGetLastError();
}

cudaError_t launch_fill_group_clip(const Launch& l, const TensorRec* tensors, uint32_t n_tensors,
                                   const float* clip, float* group_clip) {
  fill_group_clip_kernel<<<n_tensors, 256, 0, l.stream>>>(tensors, clip, group_clip);
  return cudaGetLastError();
}

// One launch over the stage's slice of the histogram tile table.  Needed whenever the stage has a
// percentile tensor: one without elements still gets its (degenerate) clip and parameters.
cudaError_t launch_hist(const Launch& l, const Stage& st, bool any16, const Tile* hist_tiles, const CalibArgs& a) {
  if (!st.any_percentile) return cudaSuccess;
  const uint32_t n_tiles = st.hist_end - st.hist_begin;
  const Tile* tp = hist_tiles + st.hist_begin;
  if (st.fused_fold) {
    const uint32_t s0 = st.any_empty ? st.tensor_begin : 0u, s1 = st.any_empty ? st.tensor_end : 0u;
    return any16 ? launch_kernel(l, hist_kernel<true, true>, st.hist_grid, kThreads, a, a.tensors, tp, n_tiles, s0, s1)
                 : launch_kernel(l, hist_kernel<false, true>, st.hist_grid, kThreads, a, a.tensors, tp, n_tiles, s0, s1);
  }
  if (n_tiles) {
    const cudaError_t e = any16
        ? launch_kernel(l, hist_kernel<true, false>, st.hist_grid, kThreads, a, a.tensors, tp, n_tiles, 0u, 0u)
        : launch_kernel(l, hist_kernel<false, false>, st.hist_grid, kThreads, a, a.tensors, tp, n_tiles, 0u, 0u);
    if (e != cudaSuccess) return e;
  }
  return launch_kernel(l, clip_fold_kernel, st.tensor_end - st.tensor_begin, kThreads, a, st.tensor_begin);
}

}  // namespace qv2
