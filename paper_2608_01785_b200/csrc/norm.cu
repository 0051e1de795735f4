// RMSNorm as a persistent, SM-budgeted kernel: one warp per token row, rows handed out in a fixed
// grid-stride order.  The sum of squares is a per-lane serial sum followed by a butterfly, so the value
// does not depend on how many blocks run.  HBM-bound: reads the row once (the second pass hits L1),
// writes the bf16 normalised row (and, for the first layer, the fp32 copy that starts the residual
// stream).
#include "kernels.h"
#include "ptx.cuh"

namespace hs {
namespace {

constexpr int NORM_THREADS = 512;
constexpr int NORM_WARPS = NORM_THREADS / 32;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void __launch_bounds__(NORM_THREADS, 1) rmsnorm_kernel(const NormParams p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int d8 = p.d >> 3;   // groups of 8 elements
  for (int row = blockIdx.x * NORM_WARPS + warp; row < p.T; row += gridDim.x * NORM_WARPS) {
    float ss = 0.f;
    if (p.x_bf16) {
      const uint4* src = reinterpret_cast<const uint4*>(p.x_bf16 + size_t(row) * p.d);
      float4* dst = reinterpret_cast<float4*>(p.x_f32_out + size_t(row) * p.d);
      for (int i = lane; i < d8; i += 32) {
        const uint4 w = src[i];
        const uint32_t u[4] = {w.x, w.y, w.z, w.w};
        float f[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          f[2 * k] = __uint_as_float(u[k] << 16);
          f[2 * k + 1] = __uint_as_float(u[k] & 0xffff0000u);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) ss += f[k] * f[k];
        dst[2 * i] = make_float4(f[0], f[1], f[2], f[3]);
        dst[2 * i + 1] = make_float4(f[4], f[5], f[6], f[7]);
      }
    } else {
      const float4* src = reinterpret_cast<const float4*>(p.x_f32 + size_t(row) * p.d);
      for (int i = lane; i < d8; i += 32) {
        const float4 a = src[2 * i], b = src[2 * i + 1];
        ss += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
        ss += b.x * b.x + b.y * b.y + b.z * b.z + b.w * b.w;
      }
    }
    ss = warp_sum(ss);
    const float r = rsqrtf(ss / float(p.d) + p.eps);
    const uint4* gsrc = reinterpret_cast<const uint4*>(p.gain);
    uint4* hdst = reinterpret_cast<uint4*>(p.h + size_t(row) * p.d);
    for (int i = lane; i < d8; i += 32) {
      float f[8];
      if (p.x_bf16) {
        const uint4 w = reinterpret_cast<const uint4*>(p.x_bf16 + size_t(row) * p.d)[i];
        const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          f[2 * k] = __uint_as_float(u[k] << 16);
          f[2 * k + 1] = __uint_as_float(u[k] & 0xffff0000u);
        }
      } else {
        const float4* src = reinterpret_cast<const float4*>(p.x_f32 + size_t(row) * p.d);
        const float4 a = src[2 * i], b = src[2 * i + 1];
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
        f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
      }
      const uint4 gw = gsrc[i];
      const uint32_t gu[4] = {gw.x, gw.y, gw.z, gw.w};
      uint32_t o[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float g0 = __uint_as_float(gu[k] << 16), g1 = __uint_as_float(gu[k] & 0xffff0000u);
        o[k] = pack_bf16(f[2 * k] * r * g0, f[2 * k + 1] * r * g1);
      }
      hdst[i] = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

}  // namespace

cudaError_t norm_set_attributes() {
  return cudaFuncSetAttribute(rmsnorm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMinSmemBytes);
}

cudaError_t launch_rmsnorm(const NormParams& p, int sm_budget, cudaStream_t stream) {
  if (p.T <= 0) return cudaSuccess;
  const int blocks = (p.T + NORM_WARPS - 1) / NORM_WARPS;
  const int grid = blocks < sm_budget ? blocks : sm_budget;
  rmsnorm_kernel<<<grid, NORM_THREADS, kMinSmemBytes, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace hs
