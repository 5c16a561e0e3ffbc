// L2 re-read probe: one persistent launch sweeps a buffer of S MB `iters` times (min/max, plain
// 16-byte loads, 8 in flight).  shift = 0: a tile is read by the same CTA every time; shift != 0: the
// CTA that reads a tile moves by `shift` blocks per iteration.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
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
template <int TILE>   // float4 per tile
__global__ void __launch_bounds__(256, 4) sweep(const float4* __restrict__ x, size_t n_vec, int iters, int shift, float2* out) {
  float mn = 1e30f, mx = -1e30f;
  const size_t n_tiles = n_vec / TILE;
  for (int it = 0; it < iters; ++it) {
    const uint32_t b = (blockIdx.x + (uint32_t)it * shift) % gridDim.x;
    for (size_t t = b; t < n_tiles; t += gridDim.x) {
      const float4* p = x + t * TILE;
      for (uint32_t j = threadIdx.x; j < TILE; j += 256 * 8) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = ld_stream4(p + j + u * 256);
#pragma unroll
        for (int u = 0; u < 8; ++u) acc4(mn, mx, v[u]);
      }
    }
  }
  if (mn > mx) out[blockIdx.x] = make_float2(mn, mx);
  if (threadIdx.x == 0 && mn == 12345.0f) out[blockIdx.x].x = mx;
}
int main() {
  int sms = 0;
  CK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0));
  const size_t maxb = 512ull << 20;
  float4* x; float2* out;
  CK(cudaMalloc(&x, maxb)); CK(cudaMalloc(&out, sizeof(float2) * sms * 8));
  CK(cudaMemset(x, 0, maxb));
  cudaEvent_t e0, e1; CK(cudaEventCreate(&e0)); CK(cudaEventCreate(&e1));
  const int grid = 4 * sms;
  printf("| MB | iters | shift | GB/s (all iterations) | us per sweep |\n|---|---|---|---|---|\n");
  for (int mb : {8, 16, 24, 32, 48, 64, 96, 128, 256, 512}) {
    for (int shift : {0, 1, grid / 2}) {
      const size_t n_vec = ((size_t)mb << 20) / 16;
      const int iters = 20;
      float best = 1e30f;
      for (int r = 0; r < 6; ++r) {
        CK(cudaEventRecord(e0));
        sweep<2048><<<grid, 256>>>(x, n_vec, iters, shift, out);
        CK(cudaEventRecord(e1));
        CK(cudaEventSynchronize(e1));
        float ms; CK(cudaEventElapsedTime(&ms, e0, e1));
        if (r >= 1) best = std::min(best, ms);
      }
      CK(cudaGetLastError());
      printf("| %d | %d | %d | %.0f | %.2f |\n", mb, iters, shift, (double)n_vec * 16 * iters / (best * 1e-3) / 1e9, best * 1e3 / iters);
    }
  }
  return 0;
}
