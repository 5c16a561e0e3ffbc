// Range calibration: one persistent launch sweeps every tile of every tensor and records the
// per-group minimum and maximum; a small second kernel turns them into absmax and quantization
// parameters (step 1 and step 2 of the paper's overview, Eq. 2 and Eq. 4).
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

// This thread's share of a flat run walked by STRIDE threads (the whole CTA, or one warp with
// tid = lane): group of four number j for j = tid, tid+STRIDE, ...; the first `head` and last
// `tail` scalars go to threads 0..2.  T is the element type in memory.
template <bool CAREFUL, uint32_t STRIDE = kThreads, class T>
__device__ __forceinline__ void range_flat(const T* __restrict__ x, uint32_t count, RangeAcc& a,
                                           uint32_t tid = threadIdx.x) {
  const FlatSplit s = split_flat(x, count);
  const T* xv = x + s.head;
  constexpr uint32_t U = sizeof(T) == 4 ? 8 : 16;       // the same bytes in flight for 16-bit types
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

// A tile of whole rows, each at least kShortRow long: one warp per row, one publication per row.
template <class T>
__device__ __forceinline__ void range_rows_tile(const T* x, const Tile& tl, const TensorRec* tr, uint32_t lane,
                                                uint32_t warp, uint32_t* kmin, uint32_t* kmax,
                                                unsigned long long* nonfinite) {
  const uint32_t inner = (uint32_t)tr->inner, channels = tr->channels;
  RangeAcc b;
  for (uint32_t r = warp; r < tl.rows; r += kWarps) {
    const T* row = x + (uint64_t)r * inner;
    reset(b);
    range_flat<false, 32>(row, inner, b, lane);
    if (__any_sync(0xffffffffu, b.nanflag != b.nanflag)) {
      reset(b);
      range_flat<true, 32>(row, inner, b, lane);
    }
    const uint32_t g = (uint32_t)((tl.row0 + r) % channels);
    publish(b, lane, kmin, kmax, tr->group_base + g, nonfinite + tl.tensor);
  }
}

// A tile of whole rows shorter than kShortRow (3x3 depthwise filters, 7x7 maps, fully connected
// activations with one element per channel): one element per thread, so that a row of nine
// elements does not occupy a warp.  Consecutive lanes hold consecutive elements; the lanes of one
// row are folded with a segmented shuffle reduction and the first lane of each run publishes.
template <class T>
__device__ __forceinline__ void range_short_rows_tile(const T* x, const Tile& tl, const TensorRec* tr,
                                                      uint32_t lane, uint32_t* kmin, uint32_t* kmax,
                                                      unsigned long long* nonfinite) {
  const uint32_t inner = (uint32_t)tr->inner, channels = tr->channels;
  const uint32_t row0c = (uint32_t)(tl.row0 % channels);
  uint32_t bad = 0;
  for (uint32_t e0 = 0; e0 < tl.count; e0 += kThreads) {        // warp-uniform bounds: every lane shuffles
    const uint32_t e = e0 + threadIdx.x;
    uint32_t row = 0xffffffffu;
    float mn = kInf, mx = -kInf;
    if (e < tl.count) {
      row = e / inner;
      const float v = Ld<T>::one(x + e);
      if (isfinite(v)) { mn = v; mx = v; } else ++bad;
    }
#pragma unroll
    for (uint32_t o = 1; o < 32; o <<= 1) {
      const float mn2 = __shfl_down_sync(0xffffffffu, mn, o), mx2 = __shfl_down_sync(0xffffffffu, mx, o);
      const uint32_t row2 = __shfl_down_sync(0xffffffffu, row, o);
      if (lane + o < 32 && row2 == row) { mn = fminf(mn, mn2); mx = fmaxf(mx, mx2); }
    }
    const uint32_t prev = __shfl_up_sync(0xffffffffu, row, 1);
    if ((lane == 0 || prev != row) && mn <= mx) {
      const uint32_t G = tr->group_base + (uint32_t)(((uint64_t)row0c + row) % channels);
      atomicMax(kmax + G, f2key(mx));
      atomicMax(kmin + G, ~f2key(mn));
    }
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
                                             uint2* rslots, unsigned long long* nonfinite_t, float* sh) {
  const float mn = warp_min(a.mn), mx = warp_max(a.mx);
  const uint32_t bad = warp_sum_u32(a.bad);
  if (lane == 0) {
    sh[warp] = mn; sh[kWarps + warp] = mx;
    if (bad) atomicAdd(nonfinite_t, (unsigned long long)bad);
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

// ANY16 = false is the build for models whose tensors are all binary32: the element-type dispatch
// is compiled out, so that common case pays nothing for the 16-bit paths.
template <bool ANY16>
__global__ void __launch_bounds__(kThreads, 4)
range_kernel(const TensorRec* __restrict__ tensors, const Tile* __restrict__ tiles, uint32_t n_tiles,
             uint32_t* kmin, uint32_t* kmax, uint2* rslots, unsigned long long* nonfinite) {
  constexpr uint32_t kNone = 0xffffffffu;
  __shared__ float sh[2 * kWarps];
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  RangeAcc a;
  reset(a);
  uint32_t cur_group = kNone, cur_tensor = 0;
  bool cur_slot = false;           // the pending group belongs to a per-tensor tensor
  for (uint32_t ti = blockIdx.x; ti < n_tiles; ti += gridDim.x) {
    const Tile tl = load_tile(tiles, ti);
    const TensorRec* tr = tensors + tl.tensor;
    const uint32_t gbase = tr->group_base;
    if (tl.rows == 0) {
      const uint32_t G = gbase + (uint32_t)tl.row0;
      if (G != cur_group) {        // block-uniform: every warp of the CTA takes this branch together
        if (cur_group != kNone) {
          if (cur_slot) publish_slot(a, lane, warp, tensors + cur_tensor, rslots, nonfinite + cur_tensor, sh);
          else publish(a, lane, kmin, kmax, cur_group, nonfinite + cur_tensor);
        }
        reset(a);
        cur_group = G; cur_tensor = tl.tensor; cur_slot = tr->per_channel == 0;
      }
      if (!ANY16 || tr->dtype == kF32) range_flat_tile(reinterpret_cast<const float*>(tr->x) + tl.begin, tl.count, a);
      else if (tr->dtype == kF16) range_flat_tile(reinterpret_cast<const __half*>(tr->x) + tl.begin, tl.count, a);
      else range_flat_tile(reinterpret_cast<const __nv_bfloat16*>(tr->x) + tl.begin, tl.count, a);
    } else if (tr->inner < kShortRow) {
      if (!ANY16 || tr->dtype == kF32)
        range_short_rows_tile(reinterpret_cast<const float*>(tr->x) + tl.begin, tl, tr, lane, kmin, kmax, nonfinite);
      else if (tr->dtype == kF16)
        range_short_rows_tile(reinterpret_cast<const __half*>(tr->x) + tl.begin, tl, tr, lane, kmin, kmax, nonfinite);
      else
        range_short_rows_tile(reinterpret_cast<const __nv_bfloat16*>(tr->x) + tl.begin, tl, tr, lane, kmin, kmax, nonfinite);
    } else {
      if (!ANY16 || tr->dtype == kF32)
        range_rows_tile(reinterpret_cast<const float*>(tr->x) + tl.begin, tl, tr, lane, warp, kmin, kmax, nonfinite);
      else if (tr->dtype == kF16)
        range_rows_tile(reinterpret_cast<const __half*>(tr->x) + tl.begin, tl, tr, lane, warp, kmin, kmax, nonfinite);
      else
        range_rows_tile(reinterpret_cast<const __nv_bfloat16*>(tr->x) + tl.begin, tl, tr, lane, warp, kmin, kmax, nonfinite);
    }
  }
  if (cur_group != kNone) {
    if (cur_slot) publish_slot(a, lane, warp, tensors + cur_tensor, rslots, nonfinite + cur_tensor, sh);
    else publish(a, lane, kmin, kmax, cur_group, nonfinite + cur_tensor);
  }
}

// One CTA per tensor: fold the CTA slots of a per-tensor tensor, decode the keys in place, write
// absmax, the tensor-wide absmax and -- for tensors without percentile clipping -- the
// quantization parameters.
// The finalize kernels are chains of dependent global loads: many threads keep the chain short
// (a tensor with 4096 groups takes 4 rounds instead of 16).
constexpr int kFinalizeThreads = 1024;

__global__ void __launch_bounds__(kFinalizeThreads)
range_finalize_kernel(const TensorRec* __restrict__ tensors, const uint2* __restrict__ rslots,
                      float* gmin, float* gmax, float* gabsmax, float* step, float* inv, float* offset,
                      float* tensor_absmax, float* clip) {
  __shared__ float red[kFinalizeThreads];
  __shared__ uint32_t kred[2][kFinalizeThreads];
  const TensorRec tr = tensors[blockIdx.x];
  if (!tr.per_channel) {                 // keys of the single group come from the slots
    uint32_t kn = 0, kx = 0;             // both arrays hold "larger is better" keys, 0 = empty
    for (uint32_t k = threadIdx.x; k < tr.rslot_count; k += blockDim.x) {
      const uint2 v = rslots[tr.rslot_first + k];
      kn = max(kn, v.x); kx = max(kx, v.y);
    }
    kred[0][threadIdx.x] = kn; kred[1][threadIdx.x] = kx;
    __syncthreads();
    for (uint32_t o = kFinalizeThreads / 2; o > 0; o >>= 1) {
      if (threadIdx.x < o) {
        kred[0][threadIdx.x] = max(kred[0][threadIdx.x], kred[0][threadIdx.x + o]);
        kred[1][threadIdx.x] = max(kred[1][threadIdx.x], kred[1][threadIdx.x + o]);
      }
      __syncthreads();
    }
    if (threadIdx.x == 0) {
      reinterpret_cast<uint32_t*>(gmin)[tr.group_base] = kred[0][0];
      reinterpret_cast<uint32_t*>(gmax)[tr.group_base] = kred[1][0];
    }
    __syncthreads();
  }
  float amax = 0.0f;
  for (uint32_t g = threadIdx.x; g < tr.n_groups; g += blockDim.x) {
    const uint32_t G = tr.group_base + g;
    const uint32_t kn = reinterpret_cast<uint32_t*>(gmin)[G];
    const uint32_t kx = reinterpret_cast<uint32_t*>(gmax)[G];
    float mn = kn ? key2f(~kn) : 0.0f;
    float mx = kx ? key2f(kx) : 0.0f;
    mn = __fadd_rn(mn, 0.0f);           // -0 -> +0, every other value unchanged
    mx = __fadd_rn(mx, 0.0f);
    const float am = fmaxf(fabsf(mn), fabsf(mx));
    gmin[G] = mn; gmax[G] = mx; gabsmax[G] = am;
    amax = fmaxf(amax, am);
    if (tr.range_mode < QV2_PERCENTILE)      // the percentile modes set theirs once the clip is known
      make_qparams(tr.asym, top_code(tr.asym != 0, tr.bits), false, 0.0f, mn, mx, am, step + G, inv + G, offset + G);
  }
  red[threadIdx.x] = amax;
  __syncthreads();
  for (uint32_t o = kFinalizeThreads / 2; o > 0; o >>= 1) {
    if (threadIdx.x < o) red[threadIdx.x] = fmaxf(red[threadIdx.x], red[threadIdx.x + o]);
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    tensor_absmax[blockIdx.x] = red[0];
    clip[blockIdx.x] = red[0];          // the percentile pass replaces it for the tensors it clips
  }
}

// Everything a calibration pass accumulates into starts at zero: the min/max keys (0 = nothing
// seen), the non-finite counters and the per-tensor histograms.  One small kernel instead of four
// memsets: a pass over a small model is bound by the number of stream operations.
__global__ void __launch_bounds__(256)
calib_init_kernel(uint32_t* kmin, uint32_t* kmax, size_t groups, unsigned long long* nonfinite, size_t n_tensors,
                  unsigned long long* hist, size_t hist_cells) {
  const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = tid; i < groups; i += stride) { kmin[i] = 0u; kmax[i] = 0u; }
  for (size_t i = tid; i < n_tensors; i += stride) nonfinite[i] = 0ull;
  for (size_t i = tid; i < hist_cells; i += stride) hist[i] = 0ull;
}

}  // namespace

cudaError_t launch_calib_init(const Launch& l, uint32_t* kmin, uint32_t* kmax, size_t groups,
                              unsigned long long* nonfinite, size_t n_tensors, unsigned long long* hist,
                              size_t hist_cells) {
  size_t most = groups > hist_cells ? groups : hist_cells;
  if (n_tensors > most) most = n_tensors;
  size_t grid = (most + 255) / 256;
  const size_t cap = (size_t)l.sm_count * 8;
  if (grid > cap) grid = cap;
  if (grid < 1) grid = 1;
  calib_init_kernel<<<(unsigned)grid, 256, 0, l.stream>>>(kmin, kmax, groups, nonfinite, n_tensors, hist, hist_cells);
  return cudaGetLastError();
}

uint32_t range_grid_cap(int sm_count) {
  static int per_sm = 0;
  return (uint32_t)persistent_grid((const void*)range_kernel<false>, &per_sm, sm_count, 0x7fffffffu);
}

cudaError_t launch_range(const Launch& l, uint32_t grid, bool any16, const TensorRec* tensors, const Tile* tiles,
                         uint32_t n_tiles, uint32_t* kmin, uint32_t* kmax, uint2* rslots,
                         unsigned long long* nonfinite) {
  if (n_tiles == 0) return cudaSuccess;
  if (any16) range_kernel<true><<<grid, kThreads, 0, l.stream>>>(tensors, tiles, n_tiles, kmin, kmax, rslots, nonfinite);
  else range_kernel<false><<<grid, kThreads, 0, l.stream>>>(tensors, tiles, n_tiles, kmin, kmax, rslots, nonfinite);
  return cudaGetLastError();
}

cudaError_t launch_range_finalize(const Launch& l, const TensorRec* tensors, uint32_t n_tensors,
                                  const uint2* rslots, float* gmin, float* gmax, float* gabsmax,
                                  float* step, float* inv, float* offset, float* tensor_absmax, float* clip) {
  range_finalize_kernel<<<n_tensors, kFinalizeThreads, 0, l.stream>>>(tensors, rslots, gmin, gmax, gabsmax, step,
                                                         inv, offset, tensor_absmax, clip);
  return cudaGetLastError();
}

}  // namespace qv2
