// |x| histogram for percentile clipping (the paper's calibration stage keeps a histogram of each
// layer's value range): 2048 linear bins on [0, absmax] per tensor, counted exactly.
//
// Each CTA keeps a private 2048 x u32 histogram in shared memory across all the tiles it walks of
// one tensor and merges it into the 64-bit global histogram only when it moves to another tensor.
// Counts are integers, so the result does not depend on the order of the atomics.
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

template <bool CAREFUL>
__device__ __forceinline__ void hist_elem(float v, float w, uint32_t* sh, uint32_t& zeros) {
  if (CAREFUL && !isfinite(v)) return;
  const uint32_t b = bin_of(v, w);
  if (b == 0) ++zeros;                 // bin 0 (half of a post-ReLU tensor) stays in a register
  else atomicAdd(sh + b, 1u);
}

template <bool CAREFUL, class T>
__device__ __forceinline__ void hist_flat(const T* __restrict__ x, uint32_t count, float w,
                                          uint32_t* sh, uint32_t& zeros) {
  const FlatSplit s = split_flat(x, count);
  const T* xv = x + s.head;
  constexpr uint32_t U = 4;
  uint32_t j = threadIdx.x;
  for (; j + (U - 1) * kThreads < s.nvec; j += U * kThreads) {
    float4 v[U];
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) v[u] = ld_vec_at(xv, j + u * kThreads);
#pragma unroll
    for (uint32_t u = 0; u < U; ++u) {
      hist_elem<CAREFUL>(v[u].x, w, sh, zeros); hist_elem<CAREFUL>(v[u].y, w, sh, zeros);
      hist_elem<CAREFUL>(v[u].z, w, sh, zeros); hist_elem<CAREFUL>(v[u].w, w, sh, zeros);
    }
  }
  for (; j < s.nvec; j += kThreads) {
    const float4 v = ld_vec_at(xv, j);
    hist_elem<CAREFUL>(v.x, w, sh, zeros); hist_elem<CAREFUL>(v.y, w, sh, zeros);
    hist_elem<CAREFUL>(v.z, w, sh, zeros); hist_elem<CAREFUL>(v.w, w, sh, zeros);
  }
  if (threadIdx.x < s.head) hist_elem<CAREFUL>(Ld<T>::one(x + threadIdx.x), w, sh, zeros);
  if (threadIdx.x < s.tail)
    hist_elem<CAREFUL>(Ld<T>::one(x + s.head + 4u * s.nvec + threadIdx.x), w, sh, zeros);
}

template <class T>
__device__ __forceinline__ void hist_tile(const T* x, uint32_t count, float w, bool careful, uint32_t* sh,
                                          uint32_t& zeros) {
  if (careful) hist_flat<true>(x, count, w, sh, zeros);
  else hist_flat<false>(x, count, w, sh, zeros);
}

template <bool ANY16>      // false: every tensor is binary32, no element-type dispatch
__global__ void __launch_bounds__(kThreads, 4)
hist_kernel(const TensorRec* __restrict__ tensors, const Tile* __restrict__ tiles, uint32_t n_tiles,
            const float* __restrict__ tensor_absmax, const unsigned long long* __restrict__ nonfinite,
            unsigned long long* hist) {
  __shared__ uint32_t sh[kBins];
  for (uint32_t b = threadIdx.x; b < kBins; b += kThreads) sh[b] = 0;
  __syncthreads();

  uint32_t cur = 0xffffffffu, since_flush = 0, zeros = 0;
  float w = 0.0f;
  bool careful = false;
  for (uint32_t ti = blockIdx.x;; ti += gridDim.x) {
    const bool more = ti < n_tiles;
    Tile tl;
    if (more) tl = load_tile(tiles, ti);
    // merge into the global histogram when the tensor changes, at the end, and before a
    // 32-bit count could overflow (2^14 tiles of 2^14 elements)
    if (cur != 0xffffffffu && (!more || tl.tensor != cur || since_flush >= 16384u)) {
      if (zeros) atomicAdd(sh, zeros);
      zeros = 0;
      __syncthreads();
      unsigned long long* h = hist + (size_t)cur * kBins;
      for (uint32_t b = threadIdx.x; b < kBins; b += kThreads) {
        const uint32_t c = sh[b];
        if (c) { atomicAdd(h + b, (unsigned long long)c); sh[b] = 0; }
      }
      __syncthreads();
      since_flush = 0;
    }
    if (!more) break;
    if (tl.tensor != cur) {
      cur = tl.tensor;
      const float A = tensor_absmax[cur];
      w = (A > 0.0f) ? __fdiv_rn((float)kBins, A) : 0.0f;
      if (!isfinite(w)) w = 0.0f;
      careful = nonfinite[cur] != 0ull;
    }
    const TensorRec* tr = tensors + cur;
    if (!ANY16 || tr->dtype == kF32) hist_tile(reinterpret_cast<const float*>(tr->x) + tl.begin, tl.count, w, careful, sh, zeros);
    else if (tr->dtype == kF16) hist_tile(reinterpret_cast<const __half*>(tr->x) + tl.begin, tl.count, w, careful, sh, zeros);
    else hist_tile(reinterpret_cast<const __nv_bfloat16*>(tr->x) + tl.begin, tl.count, w, careful, sh, zeros);
    ++since_flush;
  }
}

// One CTA per tensor: percentile clip from the histogram, then the quantization parameters of the
// tensor's groups.  T = clamp(ceil(p * Nf), 1, Nf) with Nf the histogram total; k* = first bin
// whose cumulative count reaches T; clip = upper edge of bin k* (absmax itself for the last bin).
__global__ void __launch_bounds__(256)
clip_finalize_kernel(const TensorRec* __restrict__ tensors, const unsigned long long* __restrict__ hist,
                     const float* __restrict__ tensor_absmax, const float* __restrict__ gmin,
                     const float* __restrict__ gmax, const float* __restrict__ gabsmax, float* clip,
                     float* step, float* inv, float* offset) {
  __shared__ unsigned long long scan[256];
  __shared__ uint32_t kstar_s;
  const uint32_t t = blockIdx.x, tid = threadIdx.x;
  const TensorRec tr = tensors[t];
  const float A = tensor_absmax[t];
  if (tr.range_mode != QV2_PERCENTILE) {
    if (tid == 0) clip[t] = A;
    return;
  }
  constexpr uint32_t kPer = kBins / 256;
  const unsigned long long* h = hist + (size_t)t * kBins;
  unsigned long long local[kPer], mine = 0;
#pragma unroll
  for (uint32_t i = 0; i < kPer; ++i) { local[i] = h[tid * kPer + i]; mine += local[i]; }
  scan[tid] = mine;
  if (tid == 0) kstar_s = kBins - 1;
  __syncthreads();
  for (uint32_t o = 1; o < 256; o <<= 1) {
    const unsigned long long add = tid >= o ? scan[tid - o] : 0ull;
    __syncthreads();
    scan[tid] += add;
    __syncthreads();
  }
  const unsigned long long nf = scan[255], excl = scan[tid] - mine;
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
  if (tid == 0) clip[t] = c;
  for (uint32_t g = tid; g < tr.n_groups; g += blockDim.x) {
    const uint32_t G = tr.group_base + g;
    make_qparams(tr.asym, top_code(tr.asym != 0, tr.bits), true, c, gmin[G], gmax[G], gabsmax[G], step + G, inv + G, offset + G);
  }
}

}  // namespace

cudaError_t launch_hist(const Launch& l, bool any16, const TensorRec* tensors, const Tile* tiles,
                        uint32_t n_tiles, const float* tensor_absmax,
                        const unsigned long long* nonfinite, unsigned long long* hist) {
  if (n_tiles == 0) return cudaSuccess;
  static int per_sm = 0;
  const int grid = persistent_grid((const void*)hist_kernel<false>, &per_sm, l.sm_count, n_tiles);
  if (any16) hist_kernel<true><<<grid, kThreads, 0, l.stream>>>(tensors, tiles, n_tiles, tensor_absmax, nonfinite, hist);
  else hist_kernel<false><<<grid, kThreads, 0, l.stream>>>(tensors, tiles, n_tiles, tensor_absmax, nonfinite, hist);
  return cudaGetLastError();
}

cudaError_t launch_clip_finalize(const Launch& l, const TensorRec* tensors, uint32_t n_tensors,
                                 const unsigned long long* hist, const float* tensor_absmax,
                                 const float* gmin, const float* gmax, const float* gabsmax,
                                 float* clip, float* step, float* inv, float* offset) {
  clip_finalize_kernel<<<n_tensors, 256, 0, l.stream>>>(tensors, hist, tensor_absmax, gmin, gmax,
                                                        gabsmax, clip, step, inv, offset);
  return cudaGetLastError();
}

}  // namespace qv2
