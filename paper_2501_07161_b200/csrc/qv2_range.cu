// Range calibration: one persistent launch sweeps every tile of a stage's tensors and records the
// per-group minimum and maximum; the CTA that finishes a tensor last turns them into absmax and
// quantization parameters (step 1 and step 2 of the paper's overview, Eq. 2 and Eq. 4).
//
// min/max are exact and order-independent, so the per-warp results are merged with integer
// atomicMax on an order-preserving key; no floating-point atomics are used anywhere.
#include "qv2_device.cuh"

namespace qv2 {

namespace {

constexpr float kInf = __builtin_huge_valf();

struct RangeAcc {
  float mn, mx;
  float nanflag;     // fast path: becomes NaN as soon as a non-finite element is seen
  uint32_t bad;      // careful path: count of non-finite elements
};

template <bool CAREFUL>
__device__ __forceinline__ void range_acc(RangeAcc& a, float v) {
  if (CAREFUL) {
    if (isfinite(v)) { a.mn = fminf(a.mn, v); a.mx = fmaxf(a.mx, v); }
    else ++a.bad;
  } else {
    a.mn = fminf(a.mn, v);
    a.mx = fmaxf(a.mx, v);
    a.nanflag = __fmaf_rn(v, 0.0f, a.nanflag);   // NaN*0 and Inf*0 are NaN
  }
}
template <bool CAREFUL>
__device__ __forceinline__ void range_acc4(RangeAcc& a, const float4& v) {
  range_acc<CAREFUL>(a, v.x); range_acc<CAREFUL>(a, v.y);
  range_acc<CAREFUL>(a, v.z); range_acc<CAREFUL>(a, v.w);
}

// 16-bit elements, fast path: minimum, maximum and the non-finite detector are taken two elements
// per instruction in the storage format itself (minimum and maximum are exact in any format, and
// v*0 is NaN for a NaN or an infinity in any format), and widened to binary32 once per run.
template <class T> struct Packed2;
template <> struct Packed2<__half> {
  using type = __half2;
  static __device__ __forceinline__ type both(unsigned short bits) { return __half2half2(__ushort_as_half(bits)); }
  static constexpr unsigned short kPosInf = 0x7c00u, kNegInf = 0xfc00u;
};
template <> struct Packed2<__nv_bfloat16> {
  using type = __nv_bfloat162;
  static __device__ __forceinline__ type both(unsigned short bits) {
    return __bfloat162bfloat162(__ushort_as_bfloat16(bits));
  }
  static constexpr unsigned short kPosInf = 0x7f80u, kNegInf = 0xff80u;
};

template <uint32_t STRIDE, class T>
__device__ __forceinline__ void range_flat_packed(const T* __restrict__ x, uint32_t count, RangeAcc& a, uint32_t tid) {
  using P = Packed2<T>;
  using V = typename P::type;
  const FlatSplit s = split_flat(x, count);
  const T* xv = x + s.head;
  constexpr uint32_t U = 16;                             // 8-byte loads: the same bytes in flight as 8 x 16
  V mn = P::both(P::kPosInf), mx = P::both(P::kNegInf), flag = P::both(0), zero = P::both(0);
  auto take = [&](const uint2& r) {
    const V v0 = *reinterpret_cast<const V*>(&r.x), v1 = *reinterpret_cast<const V*>(&r.y);
    mn = __hmin2(mn, v0); mx = __hmax2(mx, v0); flag = __hfma2(v0, zero, flag);
    mn = __hmin2(mn, v1); mx = __hmax2(mx, v1); flag = __hfma2(v1, zero, flag);
  };
  uint32_t j = tid;
  for (; j + (U - 1) * STRIDE < s.nvec; j += U * STRIDE) {
    uint2 r[U];
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) r[u] = ld_stream_u2(xv + 4 * (size_t)(j + u * STRIDE));
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) take(r[u]);
  }
  if (j < s.nvec) {                 // at most U-1 groups are left for this thread: one predicated round
    uint2 r[U - 1];
#pragma unroll
    for (uint32_t u = 0; u < U - 1; ++u) r[u] = ld_stream_u2(xv + 4 * (size_t)min(j + u * STRIDE, s.nvec - 1u));
#pragma unroll
    for (uint32_t u = 0; u < U - 1; ++u)
      if (j + u * STRIDE < s.nvec) take(r[u]);
  }
  a.mn = fminf(a.mn, fminf((float)mn.x, (float)mn.y));
  a.mx = fmaxf(a.mx, fmaxf((float)mx.x, (float)mx.y));
  a.nanflag = __fadd_rn(a.nanflag, __fadd_rn((float)flag.x, (float)flag.y));     // NaN if any element was not finite
  if (tid < s.head) range_acc<false>(a, Ld<T>::one(x + tid));
  if (tid < s.tail) range_acc<false>(a, Ld<T>::one(x + s.head + 4u * s.nvec + tid));
}

// This thread's share of a flat run walked by STRIDE threads (the whole CTA, or one warp with
// tid = lane): group of four number j for j = tid, tid+STRIDE, ...; the first `head` and last
// `tail` scalars go to threads 0..2.  T is the element type in memory.
// (The loop bound is per thread here: the lanes that still have a full set of groups run one more
// round before the predicated one.  The metrics and histogram walkers use the same trip count for
// every lane, which saves them a quarter of their instructions on short pieces; this kernel issues
// three instructions per element and is not bound by them, and in a same-box A/B the per-thread
// bound was the faster one for per-channel activations -- range phase 0.600 against 0.613 ms on
// ResNet-50 shapes, 0.734 against 0.755 ms on MobileNet-v2 shapes -- and equal elsewhere.)
template <bool CAREFUL, uint32_t STRIDE = kThreads, class T>
__device__ __forceinline__ void range_flat(const T* __restrict__ x, uint32_t count, RangeAcc& a,
                                           uint32_t tid = threadIdx.x) {
  if constexpr (sizeof(T) == 2 && !CAREFUL) {
    range_flat_packed<STRIDE>(x, count, a, tid);
    return;
  }
  const FlatSplit s = split_flat(x, count);
  const T* xv = x + s.head;
  constexpr uint32_t U = 8;
  uint32_t j = tid;
  for (; j + (U - 1) * STRIDE < s.nvec; j += U * STRIDE) {
    float4 v[U];
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) v[u] = ld_vec_at(xv, j + u * STRIDE);
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) range_acc4<CAREFUL>(a, v[u]);
  }
  if (j < s.nvec) {                 // at most U-1 groups are left for this thread: one predicated round
    float4 v[U - 1];
#pragma unroll
    for (uint32_t u = 0; u < U - 1; ++u) v[u] = ld_vec_at(xv, min(j + u * STRIDE, s.nvec - 1u));   // in bounds, maybe unused
#pragma unroll
    for (uint32_t u = 0; u < U - 1; ++u)
      if (j + u * STRIDE < s.nvec) range_acc4<CAREFUL>(a, v[u]);
  }
  if (tid < s.head) range_acc<CAREFUL>(a, Ld<T>::one(x + tid));
  if (tid < s.tail) range_acc<CAREFUL>(a, Ld<T>::one(x + s.head + 4u * s.nvec + tid));
}

__device__ __forceinline__ void reset(RangeAcc& a) {
  a.mn = kInf; a.mx = -kInf; a.nanflag = 0.0f; a.bad = 0;
}

// Warp-level merge and publication of one group's range.
__device__ __forceinline__ void publish(RangeAcc& a, uint32_t lane, uint32_t* kmin, uint32_t* kmax,
                                        uint32_t group, unsigned long long* nonfinite_t) {
  float mn = warp_min(a.mn), mx = warp_max(a.mx);
  uint32_t bad = warp_sum_u32(a.bad);
  if (lane == 0) {
    if (mn <= mx) {                       // false only when no finite element was seen
      atomicMax(kmax + group, f2key(mx));
      atomicMax(kmin + group, ~f2key(mn));
    }
    if (bad) atomicAdd(nonfinite_t, (unsigned long long)bad);
  }
}

// One flat tile into the running accumulator; a warp that meets a NaN or Inf redoes its share
// of the tile with exact per-element checks.
template <class T>
__device__ __forceinline__ void range_flat_tile(const T* x, uint32_t count, RangeAcc& a) {
  const float mn0 = a.mn, mx0 = a.mx;
  range_flat<false>(x, count, a);
  if (__any_sync(0xffffffffu, a.nanflag != a.nanflag)) {
    a.mn = mn0; a.mx = mx0; a.nanflag = 0.0f;
    range_flat<true>(x, count, a);
  }
}

// A tile of whole rows, each at least kLaneRow long.  The tile's elements are cut into one
// contiguous chunk per warp (a multiple of four elements, so a 16-byte aligned tile stays
// aligned); a warp walks its chunk row piece by row piece and publishes each piece's range to the
// row's group.  Eight independent streams per CTA whatever the row length: a tile of two rows of
// 8000 elements keeps every warp as busy as a tile of sixty rows of 270.
template <class T>
__device__ __noinline__ void range_rows_tile(const T* x, const Tile tl, const TensorRec* tr, uint32_t lane,
                                                uint32_t warp, uint32_t* kmin, uint32_t* kmax,
                                                unsigned long long* nonfinite) {
  const uint32_t inner = (uint32_t)tr->inner, channels = tr->channels;
  const uint32_t chunk = (tl.count + 4u * kWarps - 1u) / (4u * kWarps) * 4u;
  uint32_t c0 = min(warp * chunk, tl.count);
  const uint32_t c1 = min(c0 + chunk, tl.count);
  uint32_t row = c0 / inner;
  uint32_t row_end = (row + 1u) * inner;
  uint32_t g = (uint32_t)((tl.row0 + row) % channels);
  RangeAcc b;
  while (c0 < c1) {
    const uint32_t p1 = min(c1, row_end);
    reset(b);
    range_flat<false, 32>(x + c0, p1 - c0, b, lane);
    if (__any_sync(0xffffffffu, b.nanflag != b.nanflag)) {
      reset(b);
      range_flat<true, 32>(x + c0, p1 - c0, b, lane);
    }
    publish(b, lane, kmin, kmax, tr->group_base + g, nonfinite + tl.tensor);
    c0 = p1; row_end += inner;
    if (++g == channels) g = 0;
  }
}

// Four consecutive elements through L1 (the lane-contiguous walker below comes back to the same
// 128-byte line eight times).
template <class T> struct LdCached;
template <> struct LdCached<float> {
  static __device__ __forceinline__ float4 vec(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
};
template <> struct LdCached<__half> {
  static __device__ __forceinline__ float4 vec(const __half* p) {
    const uint2 r = __ldg(reinterpret_cast<const uint2*>(p));
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&r.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&r.y));
    return make_float4(a.x, a.y, b.x, b.y);
  }
};
template <> struct LdCached<__nv_bfloat16> {
  static __device__ __forceinline__ float4 vec(const __nv_bfloat16* p) {
    const uint2 r = __ldg(reinterpret_cast<const uint2*>(p));
    return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u),
                       __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xffff0000u));
  }
};

// A tile of whole rows shorter than kLaneRow (weight rows of 1x1 and 3x3 convolutions, depthwise
// filters, 14x14 and 7x7 maps, fully connected activations with one element per channel).  Every
// thread takes 32 CONSECUTIVE elements per round (eight 16-byte loads, all in flight), walks them
// in order and keeps the running range of the row it is in; when the row ends, and at the end of
// its 32 elements, it merges that range into the row's group with the same integer atomicMax the
// other walkers use.  A row that spans several threads is merged by each of them, which costs one
// pair of atomics per 16-32 elements and needs no exchange between threads; rows of any length
// down to a single element and of any alignment take the same path.  Non-finite elements are
// tested per element here (the flat path's redo-the-warp scheme would have to hold back every
// publication until the warp has voted).  Out of line, so that the flat path keeps its registers.
// This walker runs near 2.7 TB/s.  The cap is the serial per-element walk, not the load pattern:
// coalesced loads regrouped through shared memory gave the same times, and a coalesced variant
// that reduces the run of lanes holding a row with warp votes was slower.  Below about 300
// elements per row it still beats the per-warp chunks of
// range_rows_tile (one round trip per row piece), above it does not: 32x256x196 takes 94 against
// 120 us per 257 MB, 1000x512 36 against 24 us per 82 MB.  In a same-box A/B thresholds of 320 and
// 640 gave the same times on ResNet-18/50 and MobileNet-v2 shapes, 128 and 1024 worse ones.
constexpr uint32_t kLaneRow = 320;

template <class T>
__device__ __noinline__ void range_rows_lanes(const T* x, const Tile tl, const TensorRec* tr, uint32_t lane,
                                                 uint32_t* kmin, uint32_t* kmax, unsigned long long* nonfinite) {
  const uint32_t inner = (uint32_t)tr->inner, channels = tr->channels, gbase = tr->group_base;
  const uint32_t row0c = (uint32_t)(tl.row0 % channels);
  const FlatSplit s = split_flat(x, tl.count);
  const T* xv = x + s.head;
  uint32_t bad = 0;
  auto merge = [&](uint32_t g, float mn, float mx) {
    if (mn <= mx) {                       // false only when the piece held no finite element
      atomicMax(kmax + gbase + g, f2key(mx));
      atomicMax(kmin + gbase + g, ~f2key(mn));
    }
  };
  constexpr uint32_t V = 8;               // 16-byte groups per thread and round
  for (uint32_t v0 = threadIdx.x * V; v0 < s.nvec; v0 += kThreads * V) {
    float4 val[V];
#pragma unroll
    for (uint32_t k = 0; k < V; ++k) val[k] = LdCached<T>::vec(xv + 4 * (size_t)min(v0 + k, s.nvec - 1u));   // in bounds, maybe unused
    const uint32_t nv = min(V, s.nvec - v0);
    uint32_t e = s.head + 4u * v0;        // index in the tile of this thread's first element
    const uint32_t row = e / inner;
    uint32_t next = (row + 1u) * inner;   // first element of the next row
    uint32_t g = (row0c + row) % channels;
    float mn = kInf, mx = -kInf;
    auto take = [&](float v) {
      if (e == next) {
        merge(g, mn, mx);
        mn = kInf; mx = -kInf; next += inner;
        if (++g == channels) g = 0;
      }
      if (isfinite(v)) { mn = fminf(mn, v); mx = fmaxf(mx, v); } else ++bad;
      ++e;
    };
#pragma unroll
    for (uint32_t k = 0; k < V; ++k)
      if (k < nv) { take(val[k].x); take(val[k].y); take(val[k].z); take(val[k].w); }
    merge(g, mn, mx);
  }
  // the few elements before and after the 16-byte aligned body, one per thread
  if (threadIdx.x < s.head + s.tail) {
    const uint32_t e = threadIdx.x < s.head ? threadIdx.x : s.head + 4u * s.nvec + (threadIdx.x - s.head);
    const float v = Ld<T>::one(x + e);
    if (isfinite(v)) merge((row0c + e / inner) % channels, v, v); else ++bad;
  }
  bad = warp_sum_u32(bad);
  if (lane == 0 && bad) atomicAdd(nonfinite + tl.tensor, (unsigned long long)bad);
}

// Lanes keep their min/max across consecutive tiles of the same group and merge them only when
// the group changes.  A per-tensor tensor is ONE group cut into thousands of tiles: its CTAs
// combine their warps through shared memory and store one {min,max} key pair into the CTA's own
// slot (atomics from every warp of every CTA on that single address would serialise).  Per-channel
// groups are touched by one or two CTAs each and are merged with atomics.
__device__ __forceinline__ void publish_slot(RangeAcc& a, uint32_t lane, uint32_t warp, const TensorRec* tr,
                                             uint2* rslots, unsigned long long* nf_acc_t, float* sh) {
  const float mn = warp_min(a.mn), mx = warp_max(a.mx);
  const uint32_t bad = warp_sum_u32(a.bad);
  if (lane == 0) {
    sh[warp] = mn; sh[kWarps + warp] = mx;
    if (bad) atomicAdd(nf_acc_t, (unsigned long long)bad);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float m0 = sh[0], m1 = sh[kWarps];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) { m0 = fminf(m0, sh[w]); m1 = fmaxf(m1, sh[kWarps + w]); }
    const uint32_t g = gridDim.x;
    const uint32_t rank = (blockIdx.x + g - tr->tile_first % g) % g;
    // 0 = "no finite element seen" (m0 > m1 only in that case)
    rslots[tr->rslot_first + rank] = (m0 <= m1) ? make_uint2(~f2key(m0), f2key(m1)) : make_uint2(0u, 0u);
  }
  __syncthreads();
}

// Folds one tensor once every CTA that owns a tile of it has published: decodes the keys, writes
// min / max / absmax per group, the tensor-wide absmax, the default clip, the non-finite count
// and -- for tensors without percentile clipping -- the quantization parameters; then puts every
// accumulator it consumed back to zero, so that the next pass needs no clearing launch.  Runs in
// the CTA that drew the tensor's last ticket (or in CTA 0 for a tensor without elements); values
// written by other CTAs are read through L2.
__device__ __noinline__ void range_fold_tensor(const CalibArgs& a, uint32_t t) {
  __shared__ float red[kThreads];
  __shared__ uint32_t kred[2][kThreads];
  const TensorRec tr = a.tensors[t];
  const uint32_t tid = threadIdx.x;
  if (!tr.per_channel) {                 // keys of the single group come from the CTA slots
    uint32_t kn = 0, kx = 0;             // both hold "larger is better" keys, 0 = empty
    for (uint32_t k = tid; k < tr.range_ctas; k += kThreads) {
      const uint2 v = __ldcg(a.rslots + tr.rslot_first + k);
      kn = max(kn, v.x); kx = max(kx, v.y);
    }
    kred[0][tid] = kn; kred[1][tid] = kx;
    __syncthreads();
    for (uint32_t o = kThreads / 2; o > 0; o >>= 1) {
      if (tid < o) {
        kred[0][tid] = max(kred[0][tid], kred[0][tid + o]);
        kred[1][tid] = max(kred[1][tid], kred[1][tid + o]);
      }
      __syncthreads();
    }
  }
  float amax = 0.0f;
  for (uint32_t g = tid; g < tr.n_groups; g += kThreads) {
    const uint32_t G = tr.group_base + g;
    uint32_t kn, kx;
    if (tr.per_channel) {
      kn = __ldcg(a.kmin + G); kx = __ldcg(a.kmax + G);
      a.kmin[G] = 0u; a.kmax[G] = 0u;                  // ready for the next pass
    } else {
      kn = kred[0][0]; kx = kred[1][0];
    }
    float mn = kn ? key2f(~kn) : 0.0f;
    float mx = kx ? key2f(kx) : 0.0f;
    mn = __fadd_rn(mn, 0.0f);           // -0 -> +0, every other value unchanged
    mx = __fadd_rn(mx, 0.0f);
    const float am = fmaxf(fabsf(mn), fabsf(mx));
    a.gmin[G] = mn; a.gmax[G] = mx; a.gabsmax[G] = am;
    amax = fmaxf(amax, am);
    if (tr.range_mode < QV2_PERCENTILE)      // the percentile modes set theirs once the clip is known
      make_qparams(tr.asym, top_code(tr.asym != 0, tr.bits), false, 0.0f, mn, mx, am, a.step + G, a.inv + G,
                   a.offset + G);
  }
  red[tid] = amax;
  __syncthreads();
  for (uint32_t o = kThreads / 2; o > 0; o >>= 1) {
    if (tid < o) red[tid] = fmaxf(red[tid], red[tid + o]);
    __syncthreads();
  }
  if (tid == 0) {
    a.tensor_absmax[t] = red[0];
    a.clip[t] = red[0];                 // the percentile pass replaces it for the tensors it clips
    a.nonfinite[t] = __ldcg(a.nf_acc + t);
    a.nf_acc[t] = 0ull;
    a.tickets[t] = 0u;
  }
  // the histogram row of a tensor that is not clipped at a per-tensor percentile reads zero
  if (a.hist && tr.range_mode != QV2_PERCENTILE) {
    unsigned long long* row = a.hist + (size_t)t * kBins;
    for (uint32_t b = tid; b < kBins; b += kThreads) row[b] = 0ull;
  }
  __syncthreads();                      // the shared arrays may be reused by the next fold
}

// Ticket protocol of the fused fold.  When a CTA has published its share of tensor t (and a
// barrier has ordered every thread's publication before thread 0), thread 0 fences and draws the
// tensor's ticket WITHOUT looking at the result; the CTA goes on with its next tensor.  At its
// next tensor boundary (or when it runs out of tiles) the CTA looks at the ticket it drew: if it
// was the last one, every other owner had published before, and this CTA folds the tensor.  The
// atomic's round trip is thus hidden behind the next tensor's stream; nobody ever waits for
// another CTA.
__device__ __forceinline__ uint32_t draw_ticket(uint32_t* ticket) {    // thread 0 only
  __threadfence();                       // the CTA's publications are visible before the ticket is
  return atomicAdd(ticket, 1u);
}
__device__ __forceinline__ void range_settle(const CalibArgs& a, uint32_t t, uint32_t drawn, uint32_t* s_last) {
  if (threadIdx.x == 0) {
    const bool last = drawn == a.tensors[t].range_ctas - 1u;
    if (last) __threadfence();
    *s_last = last;
  }
  __syncthreads();
  if (*s_last) range_fold_tensor(a, t);
}

// ANY16 = false is the build for models whose tensors are all binary32: the element-type dispatch
// is compiled out, so that common case pays nothing for the 16-bit paths.
// FOLD = true: the CTA that finishes a tensor last folds it (small stages, where a separate fold
// launch would be a visible share of the pass).  FOLD = false: the kernel only publishes, and
// range_fold_kernel follows; the main loop is then free of the fold code and of its fences.
template <bool ANY16, bool FOLD>
__global__ void __launch_bounds__(kThreads, 4)
range_kernel(const __grid_constant__ CalibArgs a, const TensorRec* __restrict__ tensors,
             const Tile* __restrict__ tiles, uint32_t n_tiles, uint32_t scan_begin, uint32_t scan_end) {
  constexpr uint32_t kNone = 0xffffffffu;
  __shared__ float sh[2 * kWarps];
  __shared__ uint32_t s_last;
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  dependency_wait();
  // tensors without elements are owned by no CTA: CTA 0 folds them (the planner asks for the
  // scan only when the stage has one)
  if (FOLD && blockIdx.x == 0)
    for (uint32_t t = scan_begin; t < scan_end; ++t)
      if (tensors[t].range_ctas == 0) range_fold_tensor(a, t);
  RangeAcc acc;
  reset(acc);
  uint32_t cur_group = kNone, cur_tensor = kNone;
  uint32_t owed = kNone, drawn = 0; // FOLD: the tensor before cur_tensor and the ticket thread 0 drew for it
  bool cur_slot = false;           // the pending group belongs to a per-tensor tensor
  auto flush_group = [&]() {
    if (cur_group == kNone) return;
    if (cur_slot) publish_slot(acc, lane, warp, tensors + cur_tensor, a.rslots, a.nf_acc + cur_tensor, sh);
    else publish(acc, lane, a.kmin, a.kmax, cur_group, a.nf_acc + cur_tensor);
    cur_group = kNone;
  };
  for (uint32_t ti = blockIdx.x; ti < n_tiles; ti += gridDim.x) {
    const Tile tl = load_tile(tiles, ti);
    const TensorRec* tr = tensors + tl.tensor;
    if (tl.tensor != cur_tensor) {   // block-uniform: every warp of the CTA takes these branches together
      if (cur_tensor != kNone) {
        flush_group();
        if (FOLD) {
          if (owed != kNone) range_settle(a, owed, drawn, &s_last);
          __syncthreads();                    // every thread's publication of cur_tensor precedes the fence
          if (threadIdx.x == 0) drawn = draw_ticket(a.tickets + cur_tensor);
          owed = cur_tensor;
        }
      }
      cur_tensor = tl.tensor;
    }
    const uint32_t gbase = tr->group_base;
    if (tl.rows == 0) {
      const uint32_t G = gbase + (uint32_t)tl.row0;
      if (G != cur_group) {
        flush_group();
        reset(acc);
        cur_group = G; cur_slot = tr->per_channel == 0;
      }
      if (!ANY16 || tr->dtype == kF32) range_flat_tile(reinterpret_cast<const float*>(tr->x) + tl.begin, tl.count, acc);
      else if (tr->dtype == kF16) range_flat_tile(reinterpret_cast<const __half*>(tr->x) + tl.begin, tl.count, acc);
      else range_flat_tile(reinterpret_cast<const __nv_bfloat16*>(tr->x) + tl.begin, tl.count, acc);
    } else if (tr->inner < kLaneRow) {
      if (!ANY16 || tr->dtype == kF32)
        range_rows_lanes(reinterpret_cast<const float*>(tr->x) + tl.begin, tl, tr, lane, a.kmin, a.kmax, a.nf_acc);
      else if (tr->dtype == kF16)
        range_rows_lanes(reinterpret_cast<const __half*>(tr->x) + tl.begin, tl, tr, lane, a.kmin, a.kmax, a.nf_acc);
      else
        range_rows_lanes(reinterpret_cast<const __nv_bfloat16*>(tr->x) + tl.begin, tl, tr, lane, a.kmin, a.kmax, a.nf_acc);
    } else {
      if (!ANY16 || tr->dtype == kF32)
        range_rows_tile(reinterpret_cast<const float*>(tr->x) + tl.begin, tl, tr, lane, warp, a.kmin, a.kmax, a.nf_acc);
      else if (tr->dtype == kF16)
        range_rows_tile(reinterpret_cast<const __half*>(tr->x) + tl.begin, tl, tr, lane, warp, a.kmin, a.kmax, a.nf_acc);
      else
        range_rows_tile(reinterpret_cast<const __nv_bfloat16*>(tr->x) + tl.begin, tl, tr, lane, warp, a.kmin, a.kmax, a.nf_acc);
    }
  }
  allow_dependents();            // this CTA has issued all its loads: the next kernel may start to launch
  if (cur_tensor != kNone) {
    flush_group();
    if (FOLD) {
      if (owed != kNone) range_settle(a, owed, drawn, &s_last);
      __syncthreads();
      if (threadIdx.x == 0) drawn = draw_ticket(a.tickets + cur_tensor);
      range_settle(a, cur_tensor, drawn, &s_last);
    }
  }
}

// One CTA per tensor of the stage: the fold, for stages whose streaming kernel does not fold.
__global__ void __launch_bounds__(kThreads)
range_fold_kernel(const __grid_constant__ CalibArgs a, uint32_t tensor_begin) {
  allow_dependents();
  dependency_wait();
  range_fold_tensor(a, tensor_begin + blockIdx.x);
}

}  // namespace

uint32_t range_grid_cap(int sm_count, bool fused) {
  int cache = 0;
  const void* k = fused ? (const void*)range_kernel<false, true> : (const void*)range_kernel<false, false>;
  return (uint32_t)persistent_grid(k, &cache, sm_count, 0x7fffffffu);
}

cudaError_t launch_range(const Launch& l, const Stage& st, bool any16, const Tile* tiles, const CalibArgs& a) {
  const uint32_t n_tiles = st.tile_end - st.tile_begin;
  const Tile* tp = tiles + st.tile_begin;
  if (st.fused_fold) {
    const uint32_t s0 = st.any_empty ? st.tensor_begin : 0u, s1 = st.any_empty ? st.tensor_end : 0u;
    return any16 ? launch_kernel(l, range_kernel<true, true>, st.range_grid, kThreads, a, a.tensors, tp, n_tiles, s0, s1)
                 : launch_kernel(l, range_kernel<false, true>, st.range_grid, kThreads, a, a.tensors, tp, n_tiles, s0, s1);
  }
  if (n_tiles) {
    const cudaError_t e = any16
        ? launch_kernel(l, range_kernel<true, false>, st.range_grid, kThreads, a, a.tensors, tp, n_tiles, 0u, 0u)
        : launch_kernel(l, range_kernel<false, false>, st.range_grid, kThreads, a, a.tensors, tp, n_tiles, 0u, 0u);
    if (e != cudaSuccess) return e;
  }
  return launch_kernel(l, range_fold_kernel, st.tensor_end - st.tensor_begin, kThreads, a, st.tensor_begin);
}

}  // namespace qv2
