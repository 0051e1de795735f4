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
  griddep_wait();
  griddep_launch_dependents();
  const int d8 = p.d >> 3;                         // groups of 8 elements
  const int cached8 = min(d8, NORM_STAGE_FLOATS / 8);
  const uint4* gsrc = reinterpret_cast<const uint4*>(p.gain);
  for (int row = blockIdx.x * NORM_WARPS + warp; row < p.T; row += gridDim.x * NORM_WARPS) {
    float ss = 0.f;
    const int src_row = p.row_index ? p.row_index[row] : row;
    const uint4* xb = reinterpret_cast<const uint4*>(p.x_bf16 + size_t(src_row) * p.d);
    const float4* xf = reinterpret_cast<const float4*>(p.x_f32 + size_t(src_row) * p.d);
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
    // shift vector of the row's sequence (the scale vector follows it), or null
    const float* shift = p.mod ? p.mod + (size_t(p.tok_seq[row]) * 6 + p.mod_which) * p.d : nullptr;
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
      float v[8] = {a.x * r * g[0], a.y * r * g[1], a.z * r * g[2], a.w * r * g[3],
                    b.x * r * g[4], b.y * r * g[5], b.z * r * g[6], b.w * r * g[7]};
      if (shift) {                                   // conditioned block: (1 + scale) and shift of the row's sequence
        const float4 s0 = reinterpret_cast<const float4*>(shift)[2 * i], s1 = reinterpret_cast<const float4*>(shift)[2 * i + 1];
        const float4 c0 = reinterpret_cast<const float4*>(shift + p.d)[2 * i], c1 = reinterpret_cast<const float4*>(shift + p.d)[2 * i + 1];
        const float sh[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
        const float sc[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = fmaf(v[e], 1.f + sc[e], sh[e]);
      }
      if (f16 && p.status) note_f16_saturation(v, p.status);
      hdst[i] = make_uint4(pack_act(v[0], v[1], f16), pack_act(v[2], v[3], f16), pack_act(v[4], v[5], f16),
                           pack_act(v[6], v[7], f16));
    }
  }
}

// The same operation with rows staged by bulk copies (the variant the launcher uses whenever two rows per
// warp fit in shared memory).  Every warp owns two row buffers and an mbarrier for each; its lane 0 asks
// the copy engine for row k + 2 as soon as the warp is done with row k, so an SM keeps up to
// 2 x warps rows (about 200 KB) in flight instead of what its threads can hold in registers.  Rows are
// handed out in the same fixed order and each row's arithmetic is the same fixed sequence (a per-lane
// serial sum over groups lane, lane + 32, ... then a butterfly), whatever the grid.
constexpr int BULK_SMEM_BUDGET = 200 * 1024;   // row buffers of one block
constexpr int BULK_MAX_WARPS = 16, BULK_MIN_WARPS = 4;

__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(smem_dst)),
               "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}

// MOD: the conditioned form (shift / scale vectors per sequence); the plain form carries none of its code.
template <bool MOD>
__global__ void __launch_bounds__(BULK_MAX_WARPS * 32, 1) rmsnorm_bulk_kernel(const NormParams p) {
  extern __shared__ __align__(128) uint8_t bulk_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  log_smid(p.smid_log);
  const bool in_bf16 = p.x_bf16 != nullptr;
  const uint32_t row_bytes = uint32_t(p.d) * (in_bf16 ? 2u : 4u);
  const uint32_t buf_bytes = uint32_t(p.d) * 4u;             // buffers are sized for fp32 rows
  uint64_t* bars = reinterpret_cast<uint64_t*>(bulk_smem);    // [n_warps][2]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2 * BULK_MAX_WARPS);
  uint8_t* bufs = bulk_smem + 512 + size_t(warp) * 2 * buf_bytes;
  uint2* gains = reinterpret_cast<uint2*>(bulk_smem + 512 + size_t(n_warps) * 2 * buf_bytes);   // [d] bf16
  for (int i = threadIdx.x; i < (p.d >> 2); i += blockDim.x) gains[i] = reinterpret_cast<const uint2*>(p.gain)[i];
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2 * n_warps; ++i) mbar_init(&bars[i], 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  __syncthreads();
  griddep_wait();                 // the gains above are weights; the rows belong to the previous kernel until here
  griddep_launch_dependents();
  uint64_t* full = bars + 2 * warp;
  const int stride = gridDim.x * n_warps, first = blockIdx.x * n_warps + warp;
  const char* src = in_bf16 ? reinterpret_cast<const char*>(p.x_bf16) : reinterpret_cast<const char*>(p.x_f32);
  auto request = [&](int k) {                                 // lane 0: row number k of this warp
    const int row = first + k * stride;
    if (row < p.T) {
      const int src_row = p.row_index ? p.row_index[row] : row;
      mbar_expect_tx(&full[k & 1], row_bytes);
      bulk_load_1d(bufs + (k & 1) * buf_bytes, src + size_t(src_row) * row_bytes, row_bytes, &full[k & 1]);
    }
  };
  if (lane == 0) {
    request(0);
    request(1);
  }
  const int d4 = p.d >> 2;
  const bool f16 = p.h_f16 != 0;
  bool ok = true;
  int k = 0;
  for (int row = first; row < p.T; row += stride, ++k) {
    if (MOD) {
      // conditioned block: pull the row's shift and scale vectors (2 d floats, one after the other) into the L1
      // while the row itself is still on its way, so that the write pass below does not wait on the L2
      const char* v = reinterpret_cast<const char*>(p.mod + (size_t(p.tok_seq[row]) * 6 + p.mod_which) * p.d);
      for (int off = lane * 128; off < 2 * p.d * 4; off += 32 * 128) asm volatile("prefetch.global.L1 [%0];" ::"l"(v + off));
    }
    ok = mbar_wait(&full[k & 1], (k >> 1) & 1, abort_flag, p.status);
    if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
    const uint8_t* buf = bufs + (k & 1) * buf_bytes;
    const float4* bf = reinterpret_cast<const float4*>(buf);
    const uint2* bb = reinterpret_cast<const uint2*>(buf);
    auto group = [&](int i) {                                 // elements 4i .. 4i + 3 of the row
      if (!in_bf16) return bf[i];
      const uint2 w = bb[i];
      return make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u),
                         __uint_as_float(w.y << 16), __uint_as_float(w.y & 0xffff0000u));
    };
    // four independent partial sums per lane (groups i, i + 32, i + 64, i + 96 of every 128), combined in
    // a fixed order: enough independent work per lane to cover the shared-memory latency
    float s4[4] = {0.f, 0.f, 0.f, 0.f};
    for (int i0 = lane; i0 < d4; i0 += 128) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + 32 * u;
        if (i < d4) {
          const float4 a = group(i);
          s4[u] += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w;
        }
      }
    }
    const float ss = warp_sum((s4[0] + s4[1]) + (s4[2] + s4[3]));
    const float r = rsqrtf(ss / float(p.d) + p.eps);
    uint2* hdst = reinterpret_cast<uint2*>(p.h + size_t(row) * p.d);
    // shift vector of the row's sequence (the scale vector follows it), or null
    const float* shift = MOD ? p.mod + (size_t(p.tok_seq[row]) * 6 + p.mod_which) * p.d : nullptr;
    float4* xo = reinterpret_cast<float4*>(p.x_f32_out + size_t(row) * p.d);
    for (int i0 = lane; i0 < d4; i0 += 128) {
      float4 a[4];
      uint2 gw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + 32 * u;
        if (i < d4) {
          a[u] = group(i);
          gw[u] = gains[i];
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + 32 * u;
        if (i < d4) {
          const float g0 = __uint_as_float(gw[u].x << 16), g1 = __uint_as_float(gw[u].x & 0xffff0000u);
          const float g2 = __uint_as_float(gw[u].y << 16), g3 = __uint_as_float(gw[u].y & 0xffff0000u);
          float4 v = make_float4(a[u].x * r * g0, a[u].y * r * g1, a[u].z * r * g2, a[u].w * r * g3);
          if (MOD) {                                 // conditioned block: (1 + scale) and shift of the row's sequence
            const float4 sh = reinterpret_cast<const float4*>(shift)[i], sc = reinterpret_cast<const float4*>(shift + p.d)[i];
            v = make_float4(fmaf(v.x, 1.f + sc.x, sh.x), fmaf(v.y, 1.f + sc.y, sh.y), fmaf(v.z, 1.f + sc.z, sh.z),
                            fmaf(v.w, 1.f + sc.w, sh.w));
          }
          if (f16) {
            const float v4[4] = {v.x, v.y, v.z, v.w};
            note_f16_saturation(v4, p.status);
          }
          hdst[i] = make_uint2(pack_act(v.x, v.y, f16), pack_act(v.z, v.w, f16));
          if (in_bf16) xo[i] = a[u];                          // the widened copy that starts the residual stream
        }
      }
    }
    __syncwarp();                                             // every lane has read the buffer
    if (lane == 0) request(k + 2);
  }
  if (!ok) drain_after_abort();
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
  cudaError_t e = set_kernel_smem(rmsnorm_kernel, NORM_SMEM);
  if (e != cudaSuccess) return e;
  if ((e = set_kernel_smem(rmsnorm_bulk_kernel<false>, 512 + BULK_SMEM_BUDGET)) != cudaSuccess) return e;
  return set_kernel_smem(rmsnorm_bulk_kernel<true>, 512 + BULK_SMEM_BUDGET);
}

cudaError_t launch_rmsnorm(const NormParams& p, int sm_budget, cudaStream_t stream) {
  if (p.T <= 0) return cudaSuccess;
  // bulk-staged variant: as many warps as have room for two fp32 rows each (a function of d alone, never of
  // the budget); rows too wide for four warps fall back to the register-staged kernel
  const size_t pair_bytes = size_t(p.d) * 4 * 2, gain_bytes = size_t(p.d) * 2;
  int warps = int((BULK_SMEM_BUDGET - gain_bytes) / pair_bytes);
  if (warps > BULK_MAX_WARPS) warps = BULK_MAX_WARPS;
  if (warps >= BULK_MIN_WARPS && p.status) {
    const int blocks = (p.T + warps - 1) / warps;
    const int grid = blocks < sm_budget ? blocks : sm_budget;
    const size_t smem = 512 + size_t(warps) * pair_bytes + gain_bytes;
    const size_t bytes = smem < size_t(kMinSmemBytes) ? size_t(kMinSmemBytes) : smem;
    if (p.mod) return launch_step_kernel(rmsnorm_bulk_kernel<true>, grid, warps * 32, bytes, stream, p.overlap != 0, p);
    return launch_step_kernel(rmsnorm_bulk_kernel<false>, grid, warps * 32, bytes, stream, p.overlap != 0, p);
  }
  const int blocks = (p.T + NORM_WARPS - 1) / NORM_WARPS;
  const int grid = blocks < sm_budget ? blocks : sm_budget;
  return launch_step_kernel(rmsnorm_kernel, grid, NORM_THREADS, NORM_SMEM, stream, p.overlap != 0, p);
}

}  // namespace hs
