// Kernels of the two ends of a stage: the embedding lookup in front of hs_stage_step and greedy sampling
// (row-wise argmax of the logits) behind it.  Both are SM-budgeted like every other kernel of the library:
// persistent grids of at most sm_budget blocks that ask for more than half of an SM's shared memory, so one
// block per SM, and a fixed order of every comparison, so the result does not depend on the budget.
#include "kernels.h"
#include "ptx.cuh"

namespace hs {
namespace {

constexpr int HEAD_THREADS = 512;

// x_out[t, :] = table[tokens[t], :]: one warp per row, 16-byte loads and stores.  An id outside the table
// yields zeros and flags the status word.
__global__ void __launch_bounds__(HEAD_THREADS, 1) embed_kernel(const EmbedParams p) {
  extern __shared__ uint8_t unused_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, warps = blockDim.x >> 5;
  griddep_wait();
  griddep_launch_dependents();
  const int d8 = p.d >> 3;
  for (int t = blockIdx.x * warps + warp; t < p.n; t += gridDim.x * warps) {
    const int id = p.tokens[t];
    const bool ok = id >= 0 && id < p.vocab;
    if (!ok && lane == 0) atomicExch(p.status, kErrInvalidArg);
    const uint4* src = reinterpret_cast<const uint4*>(p.table + size_t(ok ? id : 0) * p.d);
    uint4* dst = reinterpret_cast<uint4*>(p.x_out + size_t(t) * p.d);
    for (int i = lane; i < d8; i += 32) dst[i] = ok ? src[i] : make_uint4(0, 0, 0, 0);
  }
}

// tokens[r] = lowest index of the maximum of logits[r, :].  One block per row; every thread scans a strided
// share of the row keeping (value, index) with "greater wins, on equality the lower index wins", then the
// block combines the threads' candidates with the same rule: the answer is the first maximum whatever the
// order of the combination.
__device__ __forceinline__ void take_better(float& bv, int& bi, float v, int i) {
  if (v > bv || (v == bv && i < bi)) {
    bv = v;
    bi = i;
  }
}

__global__ void __launch_bounds__(HEAD_THREADS, 1) argmax_kernel(const ArgmaxParams p) {
  extern __shared__ uint8_t argmax_smem[];
  float* sv = reinterpret_cast<float*>(argmax_smem);
  int* si = reinterpret_cast<int*>(argmax_smem + HEAD_THREADS * 4);
  griddep_wait();
  griddep_launch_dependents();
  const int v4 = p.vocab >> 2;
  for (int r = blockIdx.x; r < p.n; r += gridDim.x) {
    const float4* row = reinterpret_cast<const float4*>(p.logits + size_t(r) * p.vocab);
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    for (int i0 = threadIdx.x; i0 < v4; i0 += 4 * HEAD_THREADS) {
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (i0 + u * HEAD_THREADS < v4) v[u] = __ldcs(row + i0 + u * HEAD_THREADS);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + u * HEAD_THREADS;
        if (i < v4) {
          take_better(bv, bi, v[u].x, 4 * i);
          take_better(bv, bi, v[u].y, 4 * i + 1);
          take_better(bv, bi, v[u].z, 4 * i + 2);
          take_better(bv, bi, v[u].w, 4 * i + 3);
        }
      }
    }
    for (int i = 4 * v4 + threadIdx.x; i < p.vocab; i += HEAD_THREADS) take_better(bv, bi, p.logits[size_t(r) * p.vocab + i], i);
    sv[threadIdx.x] = bv;
    si[threadIdx.x] = bi;
    __syncthreads();
    for (int s = HEAD_THREADS / 2; s > 0; s >>= 1) {
      if (threadIdx.x < s) {
        float a = sv[threadIdx.x];
        int ai = si[threadIdx.x];
        take_better(a, ai, sv[threadIdx.x + s], si[threadIdx.x + s]);
        sv[threadIdx.x] = a;
        si[threadIdx.x] = ai;
      }
      __syncthreads();
    }
    if (threadIdx.x == 0) p.tokens[r] = si[0];
    __syncthreads();
  }
}

}  // namespace

cudaError_t head_set_attributes() {
  cudaError_t e = set_kernel_smem(embed_kernel, kMinSmemBytes);
  if (e != cudaSuccess) return e;
  return set_kernel_smem(argmax_kernel, kMinSmemBytes);
}

cudaError_t launch_embed(const EmbedParams& p, int sm_budget, cudaStream_t stream) {
  if (p.n <= 0) return cudaSuccess;
  const int warps = HEAD_THREADS / 32;
  const int blocks = (p.n + warps - 1) / warps;
  return launch_step_kernel(embed_kernel, blocks < sm_budget ? blocks : sm_budget, HEAD_THREADS, kMinSmemBytes, stream,
                            false, p);
}

cudaError_t launch_argmax(const ArgmaxParams& p, int sm_budget, cudaStream_t stream) {
  if (p.n <= 0) return cudaSuccess;
  return launch_step_kernel(argmax_kernel, p.n < sm_budget ? p.n : sm_budget, HEAD_THREADS, kMinSmemBytes, stream, false,
                            p);
}

}  // namespace hs
