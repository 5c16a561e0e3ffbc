// Read-bandwidth ceiling probe: the same min/max reduction over one large fp32 array, fed by
//  (a) plain 16-byte ld.global.nc loads with U loads in flight per thread,
//  (b) a 1-D cp.async.bulk from this GPU's own memory into one CTA's shared memory + mbarrier ring
//      with a producer warp and 8 consumer warps,
//  (c) a per-thread cp.async (16-byte LDGSTS) ring.
// Usage: read_probe [gigabytes=4] [reps=10] [only=<variant index or -1>]
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <vector>

#define CK(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("CUDA error %s at %s:%d\n", cudaGetErrorString(e_), __FILE__, __LINE__); exit(2); } } while (0)

__device__ __forceinline__ float4 ld_stream4(const float4* p) {
  float4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void acc4(float& mn, float& mx, const float4& v) {
  mn = fminf(fminf(mn, v.x), fminf(v.y, fminf(v.z, v.w)));
  mx = fmaxf(fmaxf(mx, v.x), fmaxf(v.y, fmaxf(v.z, v.w)));
}
__device__ __forceinline__ void block_out(float mn, float mx, float2* out) {
  __shared__ float smn[32], smx[32];
  for (int o = 16; o > 0; o >>= 1) { mn = fminf(mn, __shfl_xor_sync(~0u, mn, o)); mx = fmaxf(mx, __shfl_xor_sync(~0u, mx, o)); }
  if ((threadIdx.x & 31) == 0) { smn[threadIdx.x >> 5] = mn; smx[threadIdx.x >> 5] = mx; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (unsigned w = 1; w < (blockDim.x + 31) / 32; ++w) { mn = fminf(mn, smn[w]); mx = fmaxf(mx, smx[w]); }
    out[blockIdx.x] = make_float2(mn, mx);
  }
}

// (a) tiles of 16384 floats (4096 float4), CTA b takes tiles b, b+grid, ...; U loads in flight per thread
template <int U>
__global__ void __launch_bounds__(256) plain_kernel(const float4* __restrict__ x, size_t n_vec, float2* out) {
  constexpr uint32_t TILE = 4096;
  float mn = __builtin_huge_valf(), mx = -__builtin_huge_valf();
  const size_t n_tiles = n_vec / TILE;
  for (size_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
    const float4* p = x + t * TILE;
    for (uint32_t j = threadIdx.x; j < TILE; j += 256 * U) {
      float4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) v[u] = ld_stream4(p + j + u * 256);
#pragma unroll
      for (int u = 0; u < U; ++u) acc4(mn, mx, v[u]);
    }
  }
  block_out(mn, mx, out);
}

// (a') the same loads, but CTA b walks one contiguous run of tiles [b*n/g, (b+1)*n/g) instead of every g-th tile
template <int U>
__global__ void __launch_bounds__(256) plain_blocked_kernel(const float4* __restrict__ x, size_t n_vec, float2* out) {
  constexpr uint32_t TILE = 4096;
  float mn = __builtin_huge_valf(), mx = -__builtin_huge_valf();
  const size_t n_tiles = n_vec / TILE;
  const size_t t0 = n_tiles * blockIdx.x / gridDim.x, t1 = n_tiles * (blockIdx.x + 1) / gridDim.x;
  for (size_t t = t0; t < t1; ++t) {
    const float4* p = x + t * TILE;
    for (uint32_t j = threadIdx.x; j < TILE; j += 256 * U) {
      float4 v[U];
#pragma unroll
      for (int u = 0; u < U; ++u) v[u] = ld_stream4(p + j + u * 256);
#pragma unroll
      for (int u = 0; u < U; ++u) acc4(mn, mx, v[u]);
    }
  }
  block_out(mn, mx, out);
}

// ---------------------------------------------------------------------------------- mbarrier helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
// bounded wait: false when the limit ran out
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity) {
  for (uint32_t it = 0; it < (1u << 20); ++it) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* b) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(b)) : "memory");
}

// (b) producer warp + 8 consumer warps, STAGES stages of STAGE_BYTES each
template <int STAGES, int STAGE_BYTES>
__global__ void __launch_bounds__(288) bulk_kernel(const float4* __restrict__ x, size_t n_vec, float2* out, int* err) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ uint64_t full[STAGES], empty[STAGES];
  constexpr uint32_t VEC = STAGE_BYTES / 16;
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 8); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const size_t n_chunks = n_vec / VEC;
  const size_t mine = blockIdx.x < n_chunks ? (n_chunks - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  float mn = __builtin_huge_valf(), mx = -__builtin_huge_valf();
  if (warp == 0) {
    if (lane == 0) {
      size_t issued = 0;
      bool ok = true;
      for (size_t it = 0; it < mine && ok; ++it) {
        const int s = (int)(it % STAGES);
        if (it >= (size_t)STAGES) ok = mbar_wait(&empty[s], (uint32_t)((it / STAGES - 1) & 1));
        if (!ok) break;
        mbar_expect_tx(&full[s], STAGE_BYTES);
        bulk_load(smem + (size_t)s * STAGE_BYTES, x + (blockIdx.x + it * gridDim.x) * (size_t)VEC, STAGE_BYTES, &full[s]);
        ++issued;
      }
      if (!ok) {
        atomicExch(err, 1);
        // drain own copies in flight (bounded): the last min(issued, STAGES) stages
        for (size_t k = issued > (size_t)STAGES ? issued - STAGES : 0; k < issued; ++k)
          mbar_wait(&full[k % STAGES], (uint32_t)((k / STAGES) & 1));
      }
    }
  } else {
    const uint32_t ctid = threadIdx.x - 32;    // 0..255
    for (size_t it = 0; it < mine; ++it) {
      const int s = (int)(it % STAGES);
      if (!mbar_wait(&full[s], (uint32_t)((it / STAGES) & 1))) { atomicExch(err, 2); break; }
      const float4* p = reinterpret_cast<const float4*>(smem + (size_t)s * STAGE_BYTES);
#pragma unroll
      for (uint32_t j = 0; j < VEC / 256; ++j) acc4(mn, mx, p[ctid + j * 256]);
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
    }
  }
  block_out(mn, mx, out);
}

// (c) per-thread cp.async ring: each thread keeps S 16-byte copies in flight into its own slots
template <int S>
__global__ void __launch_bounds__(256) cpasync_kernel(const float4* __restrict__ x, size_t n_vec, float2* out) {
  __shared__ float4 ring[S][256];
  constexpr uint32_t TILE = 4096;
  float mn = __builtin_huge_valf(), mx = -__builtin_huge_valf();
  const size_t n_tiles = n_vec / TILE;
  // flatten this CTA's work into a sequence of float4 indices: tile t, j = tid + k*256, k < 16
  const size_t my_tiles = blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  const size_t total = my_tiles * 16;
  auto addr = [&](size_t q) { return x + (blockIdx.x + (q / 16) * gridDim.x) * (size_t)TILE + threadIdx.x + (q % 16) * 256; };
  size_t issued = 0;
  for (; issued < (size_t)(S - 1) && issued < total; ++issued) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(&ring[issued % S][threadIdx.x])), "l"(addr(issued)) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  for (size_t q = 0; q < total; ++q) {
    if (issued < total) {
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(&ring[issued % S][threadIdx.x])), "l"(addr(issued)) : "memory");
      ++issued;
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group %0;" ::"n"(S - 1) : "memory");
    acc4(mn, mx, ring[q % S][threadIdx.x]);
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  block_out(mn, mx, out);
}

struct Variant {
  const char* name;
  int grid_per_sm;
  void (*launch)(int grid, const float4* x, size_t n_vec, float2* out, int* err);
  size_t smem;
};

template <int U> void launch_plain(int grid, const float4* x, size_t n, float2* out, int*) { plain_kernel<U><<<grid, 256>>>(x, n, out); }
template <int U> void launch_plain_blocked(int grid, const float4* x, size_t n, float2* out, int*) { plain_blocked_kernel<U><<<grid, 256>>>(x, n, out); }
template <int S, int B> void launch_bulk(int grid, const float4* x, size_t n, float2* out, int* err) {
  static bool set = false;
  if (!set) { CK(cudaFuncSetAttribute(bulk_kernel<S, B>, cudaFuncAttributeMaxDynamicSharedMemorySize, S * B)); set = true; }
  bulk_kernel<S, B><<<grid, 288, S * B>>>(x, n, out, err);
}
template <int S> void launch_cpasync(int grid, const float4* x, size_t n, float2* out, int*) { cpasync_kernel<S><<<grid, 256>>>(x, n, out); }

int main(int argc, char** argv) {
  const double gb = argc > 1 ? atof(argv[1]) : 4.0;
  const int reps = argc > 2 ? atoi(argv[2]) : 10;
  const int only = argc > 3 ? atoi(argv[3]) : -1;
  size_t n_vec = (size_t)(gb * (1ull << 30)) / 16;
  n_vec = n_vec / 65536 * 65536;                 // whole tiles and whole stages for every variant
  const size_t bytes = n_vec * 16;
  int sms = 0;
  CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
  float4* x; float2* out; int* err;
  CK(cudaMalloc(&x, bytes));
  CK(cudaMalloc(&out, sizeof(float2) * sms * 16));
  CK(cudaMalloc(&err, sizeof(int)));
  CK(cudaMemset(err, 0, sizeof(int)));
  {  // fill with a cheap pattern: floats in (-1, 1), with planted extremes
    std::vector<float> h(1 << 22);
    uint32_t s = 12345u;
    for (auto& v : h) { s = s * 1664525u + 1013904223u; v = ((s >> 8) / 8388608.0f) - 1.0f; }
    for (size_t off = 0; off < bytes; off += h.size() * 4) CK(cudaMemcpy((char*)x + off, h.data(), std::min(h.size() * 4, bytes - off), cudaMemcpyHostToDevice));
    float lo = -3.5f, hi = 7.25f;
    CK(cudaMemcpy((char*)x + bytes / 3 / 16 * 16, &lo, 4, cudaMemcpyHostToDevice));
    CK(cudaMemcpy((char*)x + bytes - 4, &hi, 4, cudaMemcpyHostToDevice));
  }
  std::vector<Variant> vs = {
      {"plain ld.global.nc.v4, 4 in flight, 8 CTA/SM", 8, launch_plain<4>, 0},
      {"plain ld.global.nc.v4, 8 in flight, 4 CTA/SM", 4, launch_plain<8>, 0},
      {"plain ld.global.nc.v4, 8 in flight, 8 CTA/SM", 8, launch_plain<8>, 0},
      {"plain ld.global.nc.v4, 16 in flight, 4 CTA/SM", 4, launch_plain<16>, 0},
      {"cp.async.bulk ring 4 x 16 KB, 3 CTA/SM", 3, launch_bulk<4, 16384>, 4 * 16384},
      {"cp.async.bulk ring 3 x 32 KB, 2 CTA/SM", 2, launch_bulk<3, 32768>, 3 * 32768},
      {"cp.async.bulk ring 6 x 16 KB, 2 CTA/SM", 2, launch_bulk<6, 16384>, 6 * 16384},
      {"cp.async.bulk ring 8 x 8 KB, 3 CTA/SM", 3, launch_bulk<8, 8192>, 8 * 8192},
      {"cp.async.bulk ring 6 x 32 KB, 1 CTA/SM", 1, launch_bulk<6, 32768>, 6 * 32768},
      {"cp.async 16 B per thread, 4 stages, 4 CTA/SM", 4, launch_cpasync<4>, 0},
      {"cp.async 16 B per thread, 8 stages, 4 CTA/SM", 4, launch_cpasync<8>, 0},
      {"plain ld.global.nc.v4, 8 in flight, 4 CTA/SM, one contiguous run of tiles per CTA", 4, launch_plain_blocked<8>, 0},
      {"plain ld.global.nc.v4, 8 in flight, 3 CTA/SM, one contiguous run of tiles per CTA", 3, launch_plain_blocked<8>, 0},
      {"plain ld.global.nc.v4, 8 in flight, 3 CTA/SM", 3, launch_plain<8>, 0},
  };
  cudaEvent_t e0, e1;
  CK(cudaEventCreate(&e0)); CK(cudaEventCreate(&e1));
  printf("input %.3f GB, %d SMs, %d reps per variant\n", bytes / 1e9, sms, reps);
  printf("| variant | best GB/s | median GB/s | min | max |\n|---|---|---|---|---|\n");
  for (size_t vi = 0; vi < vs.size(); ++vi) {
    if (only >= 0 && (int)vi != only) continue;
    const Variant& v = vs[vi];
    const int grid = v.grid_per_sm * sms;
    for (int w = 0; w < 2; ++w) v.launch(grid, x, n_vec, out, err);
    CK(cudaGetLastError());
    CK(cudaDeviceSynchronize());
    std::vector<float> ms(reps);
    for (int r = 0; r < reps; ++r) {
      CK(cudaEventRecord(e0));
      v.launch(grid, x, n_vec, out, err);
      CK(cudaEventRecord(e1));
      CK(cudaEventSynchronize(e1));
      CK(cudaEventElapsedTime(&ms[r], e0, e1));
    }
    CK(cudaGetLastError());
    std::vector<float2> h(grid);
    int herr = 0;
    CK(cudaMemcpy(h.data(), out, sizeof(float2) * grid, cudaMemcpyDeviceToHost));
    CK(cudaMemcpy(&herr, err, sizeof(int), cudaMemcpyDeviceToHost));
    float mn = 1e30f, mx = -1e30f;
    for (auto& p : h) { mn = std::min(mn, p.x); mx = std::max(mx, p.y); }
    std::sort(ms.begin(), ms.end());
    printf("| %s | %.0f | %.0f | %g | %g |%s\n", v.name, bytes / (ms[0] * 1e-3) / 1e9, bytes / (ms[reps / 2] * 1e-3) / 1e9, mn, mx,
           (herr || mn != -3.5f || mx != 7.25f) ? " WRONG" : "");
    if (herr) { printf("wait limit ran out (err=%d)\n", herr); return 3; }
  }
  return 0;
}
