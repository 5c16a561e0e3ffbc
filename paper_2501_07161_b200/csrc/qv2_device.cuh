// Device helpers shared by the streaming kernels: streaming loads, the tile fetch, the split of
// a flat element run into an aligned 16-byte body with scalar head/tail, and warp reductions.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "qv2_common.cuh"

namespace qv2 {

// Programmatic dependent launch.  dependency_wait(): returns once the kernel this launch depends
// on has completed and its writes are visible (immediately when the launch was an ordinary one).
// allow_dependents(): the next kernel of the stream may be scheduled as soon as every CTA of this
// one has said so; its CTAs then wait in dependency_wait() for this kernel to finish.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void allow_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Read-once data: bypass L1 allocation so the stream does not evict anything useful.
__device__ __forceinline__ float4 ld_stream4(const float4* p) {
  float4 v;
  asm("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
      : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
      : "l"(p));
  return v;
}
__device__ __forceinline__ float ld_stream1(const float* p) {
  float v;
  asm("ld.global.nc.L1::no_allocate.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}

// Element access by type: four consecutive elements widened to binary32 (the address must be a
// multiple of four elements), or one element.  binary16 and bfloat16 widen exactly.
template <class T> struct Ld;
// vec_at(base, j): the j-th group of four after `base`; the index is widened before it is scaled
// so that the address is one multiply-add.
template <class T>
__device__ __forceinline__ float4 ld_vec_at(const T* base, uint32_t j) { return Ld<T>::vec(base + 4 * (size_t)j); }
template <> struct Ld<float> {
  static __device__ __forceinline__ float4 vec(const float* p) { return ld_stream4(reinterpret_cast<const float4*>(p)); }
  static __device__ __forceinline__ float one(const float* p) { return ld_stream1(p); }
};
__device__ __forceinline__ uint2 ld_stream_u2(const void* p) {
  uint2 v;
  asm("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ unsigned short ld_stream_u16(const void* p) {
  unsigned short v;
  asm("ld.global.nc.L1::no_allocate.u16 %0, [%1];" : "=h"(v) : "l"(p));
  return v;
}
template <> struct Ld<__half> {
  static __device__ __forceinline__ float4 vec(const __half* p) {
    const uint2 r = ld_stream_u2(p);
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&r.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&r.y));
    return make_float4(a.x, a.y, b.x, b.y);
  }
  static __device__ __forceinline__ float one(const __half* p) {
    return __half2float(__ushort_as_half(ld_stream_u16(p)));
  }
};
template <> struct Ld<__nv_bfloat16> {      // a bfloat16 is the upper half of a binary32
  static __device__ __forceinline__ float4 vec(const __nv_bfloat16* p) {
    const uint2 r = ld_stream_u2(p);
    return make_float4(__uint_as_float(r.x << 16), __uint_as_float(r.x & 0xffff0000u),
                       __uint_as_float(r.y << 16), __uint_as_float(r.y & 0xffff0000u));
  }
  static __device__ __forceinline__ float one(const __nv_bfloat16* p) {
    return __uint_as_float((uint32_t)ld_stream_u16(p) << 16);
  }
};

__device__ __forceinline__ Tile load_tile(const Tile* tiles, uint32_t i) {
  const uint4* p = reinterpret_cast<const uint4*>(tiles + i);
  uint4 a = __ldg(p), b = __ldg(p + 1);
  Tile t;
  t.begin = (uint64_t)a.x | ((uint64_t)a.y << 32);
  t.row0 = (uint64_t)a.z | ((uint64_t)a.w << 32);
  t.count = b.x; t.tensor = b.y; t.rows = b.z; t.pack = b.w;
  return t;
}

// A flat run [p, p+count): `head` scalars up to the first address that is a multiple of four
// elements (16 bytes of binary32, 8 of the 16-bit types), `nvec` groups of four, `tail` scalars.
struct FlatSplit {
  uint32_t head, nvec, tail;
};
template <class T>
__device__ __forceinline__ FlatSplit split_flat(const T* p, uint32_t count) {
  FlatSplit s;
  uint32_t mis = (uint32_t)(((uintptr_t)p / sizeof(T)) & 3u);   // elements past a 4-element boundary
  uint32_t head = (4u - mis) & 3u;
  s.head = head < count ? head : count;
  s.nvec = (count - s.head) >> 2;
  s.tail = count - s.head - 4u * s.nvec;
  return s;
}

__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// Butterfly sum: every lane ends with the same value and the order of additions is fixed.
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = __fadd_rn(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = __dadd_rn(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ uint32_t warp_sum_u32(uint32_t v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Order-preserving map float -> uint32 (larger float <=> larger key).  Never 0 for a non-NaN
// input, so 0 marks "nothing recorded" in the min/max key arrays.
__device__ __forceinline__ uint32_t f2key(float f) {
  uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key2f(uint32_t k) {
  uint32_t b = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
  return __uint_as_float(b);
}

// Quantization parameters of one group (Eq. 4 read as the multiplier 127/max|W|; Eq. 2 for the
// affine form), one binary32 rounding per operation.
// `top` is the largest code: 2^(b-1) - 1 (symmetric) or 2^b - 1 (affine); 127 / 255 at 8 bits.
__device__ __host__ __forceinline__ float top_code(bool asym, uint32_t bits) {
  return (float)(asym ? (1u << bits) - 1u : (1u << (bits - 1u)) - 1u);
}
// scheme: 0 symmetric, 1 affine with the real-valued minimum as offset, 2 affine with an integer
// zero point (range widened to hold 0; the offset slot then carries z = clamp(rne(-lo/step), 0, top)).
__device__ __forceinline__ void make_qparams(uint32_t scheme, float top, bool use_clip, float clip, float mn,
                                             float mx, float am, float* step, float* inv, float* offset) {
  const bool asym = scheme != 0;
  float s, r, off;
  if (!asym) {
    float R = am;
    if (use_clip && clip < R) R = clip;
    s = __fdiv_rn(R, top);
    r = __fdiv_rn(top, R);
    off = 0.0f;
    if (!(R > 0.0f) || !isfinite(r) || !(s > 0.0f)) { s = 1.0f; r = 1.0f; }
  } else {
    float lo = mn, hi = mx;
    if (use_clip) {
      if (-clip > lo) lo = -clip;
      if (clip < hi) hi = clip;
    }
    if (scheme == 2) {
      if (lo > 0.0f) lo = 0.0f;
      if (hi < 0.0f) hi = 0.0f;
    }
    lo = __fadd_rn(lo, 0.0f);            // -0 -> +0
    float d = __fsub_rn(hi, lo);
    s = __fdiv_rn(d, top);
    r = __fdiv_rn(top, d);
    off = lo;
    if (!(d > 0.0f) || !isfinite(r) || !(s > 0.0f)) {
      s = 1.0f; r = 1.0f;
      if (scheme == 2) off = 0.0f;
    } else if (scheme == 2) {
      float z = rintf(__fdiv_rn(-lo, s));          // round half to even
      if (!(z >= 0.0f)) z = 0.0f;
      off = fminf(z, top);
    }
  }
  *step = s; *inv = r; *offset = off;
}

// Grid of a persistent streaming kernel: every SM filled with as many CTAs as fit, never more
// CTAs than tiles.  `cache` keeps the occupancy answer of one kernel between launches.
inline int persistent_grid(const void* kernel, int* cache, int sm_count, uint32_t n_tiles) {
  if (*cache <= 0) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0) != cudaSuccess ||
        per_sm < 1)
      per_sm = 1;
    *cache = per_sm;
  }
  long long g = (long long)(*cache) * sm_count;
  if (g > (long long)n_tiles) g = n_tiles;
  return g < 1 ? 1 : (int)g;
}

}  // namespace qv2
