// RMSNorm as a persistent, SM-budgeted kernel: one warp per token row, rows handed out in a fixed
// grid-stride order.  The sum of squares is a per-lane serial sum followed by a butterfly, so the value
// does not depend on how many blocks run.  HBM-bound: reads the row once (it is kept in shared memory for
// the scaling pass), writes the bf16 normalised row (and, for the first layer, the fp32 copy that starts
// the residual stream).
#include "kernels.h"
#include "ptx.cuh"

namespace hs {
namespace {

constexpr int NORM_THREADS = 512;
constexpr int NORM_WARPS = NORM_THREADS / 32;
constexpr int NORM_STAGE_FLOATS = 2048;   // per-warp row cache in shared memory (rows up to this width)
constexpr int NORM_SMEM = NORM_WARPS * NORM_STAGE_FLOATS * 4 > kMinSmemBytes ? NORM_WARPS * NORM_STAGE_FLOATS * 4
                                                                              : kMinSmemBytes;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ void unpack8(const uint4& w, float (&f)[8]) {
  const uint32_t u[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    f[2 * k] = __uint_as_float(u[k] << 16);
    f[2 * k + 1] = __uint_as_float(u[k] & 0xffff0000u);
  }
}

// The row is read from global memory once: the first pass keeps it in the warp's slice of shared memory
// (rows wider than the slice fall back to a second global read of the tail), the second pass scales it.
__global__ void __launch_bounds__(NORM_THREADS, 1) rmsnorm_kernel(const NormParams p) {
  extern __shared__ float norm_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  log_smid(p.smid_log);
  float4* cache = reinterpret_cast<float4*>(norm_smem + warp * NORM_STAGE_FLOATS);
  const int d8 = p.d >> 3;                         // groups of 8 elements
  const int cached8 = min(d8, NORM_STAGE_FLOATS / 8);
  const uint4* gsrc = reinterpret_cast<const uint4*>(p.gain);
  for (int row = blockIdx.x * NORM_WARPS + warp; row < p.T; row += gridDim.x * NORM_WARPS) {
    float ss = 0.f;
    const uint4* xb = reinterpret_cast<const uint4*>(p.x_bf16 + size_t(row) * p.d);
    const float4* xf = reinterpret_cast<const float4*>(p.x_f32 + size_t(row) * p.d);
    float4* xo = reinterpret_cast<float4*>(p.x_f32_out + size_t(row) * p.d);
    // four groups per lane are requested before any is used, to keep enough bytes in flight
    for (int i0 = lane; i0 < d8; i0 += 128) {
      float4 a[4], b[4];
      if (p.x_bf16) {
        uint4 w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
          if (i0 + 32 * k < d8) w[k] = xb[i0 + 32 * k];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (i0 + 32 * k < d8) {
            float f[8];
            unpack8(w[k], f);
            a[k] = make_float4(f[0], f[1], f[2], f[3]);
            b[k] = make_float4(f[4], f[5], f[6], f[7]);
            xo[2 * (i0 + 32 * k)] = a[k];
            xo[2 * (i0 + 32 * k) + 1] = b[k];
          }
        }
      } else {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          if (i0 + 32 * k < d8) {
            a[k] = xf[2 * (i0 + 32 * k)];
            b[k] = xf[2 * (i0 + 32 * k) + 1];
          }
        }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = i0 + 32 * k;
        if (i < d8) {
          ss += a[k].x * a[k].x + a[k].y * a[k].y + a[k].z * a[k].z + a[k].w * a[k].w;
          ss += b[k].x * b[k].x + b[k].y * b[k].y + b[k].z * b[k].z + b[k].w * b[k].w;
          if (i < cached8) {
            cache[2 * i] = a[k];
            cache[2 * i + 1] = b[k];
          }
        }
      }
    }
    ss = warp_sum(ss);
    const float r = rsqrtf(ss / float(p.d) + p.eps);
    uint4* hdst = reinterpret_cast<uint4*>(p.h + size_t(row) * p.d);
    for (int i = lane; i < d8; i += 32) {
      float4 a, b;
      if (i < cached8) {                            // written by this same lane above
        a = cache[2 * i];
        b = cache[2 * i + 1];
      } else if (p.x_bf16) {
        float f[8];
        unpack8(xb[i], f);
        a = make_float4(f[0], f[1], f[2], f[3]);
        b = make_float4(f[4], f[5], f[6], f[7]);
      } else {
        a = xf[2 * i];
        b = xf[2 * i + 1];
      }
      float g[8];
      unpack8(gsrc[i], g);
      const bool f16 = p.h_f16 != 0;
      hdst[i] = make_uint4(pack_act(a.x * r * g[0], a.y * r * g[1], f16), pack_act(a.z * r * g[2], a.w * r * g[3], f16),
                           pack_act(b.x * r * g[4], b.y * r * g[5], f16), pack_act(b.z * r * g[6], b.w * r * g[7], f16));
    }
  }
}

// One-time widening of the significand: bf16 weights -> fp16 copies (n8 groups of 8 values).  A bf16 value
// is an fp16 value exactly when 2^-17 <= |w| <= 65504; smaller ones round to the fp16 subnormal grid
// (absolute error <= 2^-25), larger ones saturate.
__global__ void __launch_bounds__(256) bf16_to_f16_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                                          size_t n8) {
  for (size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x; i < n8; i += size_t(gridDim.x) * blockDim.x) {
    float f[8];
    unpack8(src[i], f);
    dst[i] = make_uint4(pack_f16(f[0], f[1]), pack_f16(f[2], f[3]), pack_f16(f[4], f[5]), pack_f16(f[6], f[7]));
  }
}

}  // namespace

cudaError_t launch_bf16_to_f16(const void* src, void* dst, size_t n, cudaStream_t stream) {
  const size_t n8 = n / 8;
  if (n8 == 0) return cudaSuccess;
  const size_t want = (n8 + 255) / 256;
  bf16_to_f16_kernel<<<unsigned(want < 1184 ? want : 1184), 256, 0, stream>>>(static_cast<const uint4*>(src),
                                                                              static_cast<uint4*>(dst), n8);
  return cudaGetLastError();
}

cudaError_t norm_set_attributes() {
  return cudaFuncSetAttribute(rmsnorm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, NORM_SMEM);
}

cudaError_t launch_rmsnorm(const NormParams& p, int sm_budget, cudaStream_t stream) {
  if (p.T <= 0) return cudaSuccess;
  const int blocks = (p.T + NORM_WARPS - 1) / NORM_WARPS;
  const int grid = blocks < sm_budget ? blocks : sm_budget;
  rmsnorm_kernel<<<grid, NORM_THREADS, NORM_SMEM, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace hs
