// Convolution + batch-normalisation folding (Eq. 10-12): the weights that the sensitivity sweep
// sees when the model is analysed on the fused graph.  A_c = gamma_c / sqrt(var_c) * W_c and
// C_c = gamma_c (B_c - mean_c) / sqrt(var_c) + beta_c, per output channel c.  A pure streaming
// pre-pass: 4 bytes read and 4 bytes written per weight.
#include "qv2_device.cuh"

namespace qv2 {

namespace {

// One binary32 rounding per operation, in this order: r = sqrt(var), s = gamma / r.
__device__ __forceinline__ float fold_scale(float gamma, float var) {
  return __fdiv_rn(gamma, __fsqrt_rn(var));
}

// grid.y = channel, grid.x * blockDim.x covers the row; VEC selects 128-bit accesses.
// INPLACE: w_out is w itself.  Every element is then read and written by the same thread, which
// is safe, but the read-only (non-coherent) load path and the no-alias promise are not: the
// in-place build uses plain loads and unqualified pointers.
template <bool VEC, bool INPLACE>
__global__ void __launch_bounds__(256)
fold_kernel(const float* w, const float* __restrict__ gamma, const float* __restrict__ var,
            uint64_t inner, float* w_out) {
  const uint64_t c = blockIdx.y;
  const float s = fold_scale(__ldg(gamma + c), __ldg(var + c));
  const float* row = w + c * inner;
  float* out = w_out + c * inner;
  if (VEC) {
    const uint64_t nvec = inner >> 2;
    for (uint64_t j = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; j < nvec; j += (uint64_t)gridDim.x * blockDim.x) {
      float4 v = INPLACE ? reinterpret_cast<const float4*>(row)[j] : ld_stream4(reinterpret_cast<const float4*>(row) + j);
      v.x = __fmul_rn(s, v.x); v.y = __fmul_rn(s, v.y); v.z = __fmul_rn(s, v.z); v.w = __fmul_rn(s, v.w);
      reinterpret_cast<float4*>(out)[j] = v;
    }
  } else {
    for (uint64_t j = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; j < inner; j += (uint64_t)gridDim.x * blockDim.x)
      out[j] = __fmul_rn(s, INPLACE ? row[j] : ld_stream1(row + j));
  }
}

__global__ void fold_bias_kernel(const float* __restrict__ bias, const float* __restrict__ gamma,
                                 const float* __restrict__ beta, const float* __restrict__ mean,
                                 const float* __restrict__ var, uint64_t channels, float* __restrict__ bias_out) {
  const uint64_t c = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x;
  if (c >= channels) return;
  const float s = fold_scale(gamma[c], var[c]);
  const float b = bias ? bias[c] : 0.0f;
  bias_out[c] = __fadd_rn(__fmul_rn(s, __fsub_rn(b, mean[c])), beta[c]);
}

}  // namespace

cudaError_t launch_fold(const Launch& l, const float* w, const float* bias, const float* gamma,
                        const float* beta, const float* mean, const float* var, uint64_t channels,
                        uint64_t inner, float* w_out, float* bias_out) {
  if (channels == 0) return cudaSuccess;
  if (inner) {
    const bool vec = (inner % 4 == 0) && ((((uintptr_t)w) | ((uintptr_t)w_out)) & 15u) == 0;
    const uint64_t per_row = vec ? inner / 4 : inner;
    uint64_t gx = (per_row + 255) / 256;
    if (gx > 64) gx = 64;
    for (uint64_t c0 = 0; c0 < channels; c0 += 65535) {       // grid.y limit
      const uint64_t nc = channels - c0 < 65535 ? channels - c0 : 65535;
      dim3 grid((unsigned)gx, (unsigned)nc);
      const float* wp = w + c0 * inner; float* op = w_out + c0 * inner;
      if (w == w_out) {
        if (vec) fold_kernel<true, true><<<grid, 256, 0, l.stream>>>(wp, gamma + c0, var + c0, inner, op);
        else fold_kernel<false, true><<<grid, 256, 0, l.stream>>>(wp, gamma + c0, var + c0, inner, op);
      } else {
        if (vec) fold_kernel<true, false><<<grid, 256, 0, l.stream>>>(wp, gamma + c0, var + c0, inner, op);
        else fold_kernel<false, false><<<grid, 256, 0, l.stream>>>(wp, gamma + c0, var + c0, inner, op);
      }
    }
  }
  if (bias_out)
    fold_bias_kernel<<<(unsigned)((channels + 255) / 256), 256, 0, l.stream>>>(bias, gamma, beta, mean, var,
                                                                              channels, bias_out);
  return cudaGetLastError();
}

}  // namespace qv2
