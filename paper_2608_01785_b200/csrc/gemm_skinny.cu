// The projections of a small step (at most 64 token rows).  With so few rows every GEMM of the layer is a
// weight-streaming problem, and what counts is how many SMs pull weights and how directly.  The tcgen05 kernel
// of gemm.cu feeds 128-row tiles through TMA boxes of 128-byte pieces and needs a K split with an ordered
// chain of adds to occupy the GPU; this kernel does the opposite:
//   * one block per unit of 32 output columns and the WHOLE K range: no K split across blocks, no chain;
//   * inside the block the K range is dealt over 8 warps; every warp streams its K steps of the unit's 32 weight
//     rows with 16-byte cp.async copies into a private ring of shared memory (every lane reads back exactly the
//     16 bytes it copied, so the ring needs no barrier at all), the matching slice of the activations the same
//     way, and feeds mma.sync m16n8k16 fragments from the ring -- no TMA, no TMEM, no mbarrier;
//   * the 8 partial accumulators meet in shared memory and are summed in warp order, then the epilogue of the
//     mode runs: residual add, RoPE + cache write + q store, or SwiGLU.
// Units are listed independently of the SM budget and a unit's arithmetic is one fixed sequence, so the results
// do not depend on the budget.  A unit's 32 columns are chosen per mode so that the epilogue finds its partner
// columns in the same thread: Qkv units take columns c .. c+15 and c + Dh/2 .. c + Dh/2 + 15 of one head (the
// rotation pairs), GateUp units 16 gate columns and the same 16 up columns.
//
// Fragment trick: a lane loads 8 consecutive K elements (16 bytes) of its weight row and of its two
// activation rows; the two MMAs of a 32-wide K step use elements 0..3 and 4..7 of those.  That is a
// permutation of the K index inside the step, applied to both operands alike, so the dot products are
// unchanged and every load is a full 16 bytes.
#include <cuda_fp16.h>

#include <algorithm>

#include "attention_decode.cuh"
#include "kernels.h"
#include "ptx.cuh"

namespace hs {
namespace {

constexpr int SK_WARPS = 8, SK_THREADS = SK_WARPS * 32;

template <bool F16>
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1) {
  if (F16)
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  else
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// cp.async.cg reads through the L2 only: right for weights that are used once and for activations that the
// kernel before this one wrote (it may still be draining when this kernel starts).
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 lds16(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}

// First element of (slot, kv head) in one layer's K or V pages: [page][kv_head][16][Dh].
__device__ __forceinline__ __nv_bfloat16* cache_row(__nv_bfloat16* base, int slot, int hk, int n_kv_heads, int Dh) {
  return base + ((size_t(slot >> 4) * n_kv_heads + hk) * 16 + (slot & 15)) * Dh;
}

constexpr int NT = 4;                  // n8 tiles of a unit: 32 output columns
constexpr int PART_STRIDE = 40;        // floats between rows of a warp's partial tile (32 + padding)

// Where tile j (0..3), column g (0..7) of unit `unit` lives: the weight row to read.
__device__ __forceinline__ const uint8_t* unit_row(const SkinnyParams& p, int unit, int j, int g) {
  const size_t row_bytes = size_t(p.K) * 2;
  if (p.mode == kGemmResid) return static_cast<const uint8_t*>(p.w[0]) + size_t(unit * 32 + j * 8 + g) * row_bytes;
  if (p.mode == kGemmGateUp) {
    const int r = unit * 16 + (j & 1) * 8 + g;                       // tiles 0,1 gate; 2,3 the same rows of up
    return static_cast<const uint8_t*>(p.w[j >> 1]) + size_t(r) * row_bytes;
  }
  const int upr = p.head_dim >> 5;                                   // units per head
  const int head = unit / upr, sub = unit - head * upr;
  int col = head * p.head_dim + sub * 16 + (j & 1) * 8 + g + (j >> 1) * (p.head_dim >> 1);
  int which = 0;
  if (col >= p.q_dim) { col -= p.q_dim; which = 1; }
  if (which == 1 && col >= p.kv_dim) { col -= p.kv_dim; which = 2; }
  return static_cast<const uint8_t*>(p.w[which]) + size_t(col) * row_bytes;
}


// MT: 16-row tiles of activations (T <= 16 MT); DB: depth of a warp's ring of K steps.
// FOLD: the instantiation that knows the folded RMSNorm (producing side in Resid mode, consuming side in the others);
// the plain one carries none of its code.
// r = rsqrt(mean(x^2) + eps) of row `row` from its n partial sums of squares (one per 32 columns): the four threads
// of a row (threadIdx & 3) add every fourth partial each and then combine, a fixed order whoever calls.  Called by all
// threads of a warp.
__device__ __forceinline__ float row_norm_factor(const float* row_ss, int stride, int n, int row, int T, int width, float eps) {
  const int q = threadIdx.x & 3;
  float sum = 0.f;
  if (row < T)
    for (int i = q; i < n; i += 4) sum += __ldcg(row_ss + size_t(row) * stride + i);
  sum += __shfl_xor_sync(0xffffffffu, sum, 1);
  sum += __shfl_xor_sync(0xffffffffu, sum, 2);
  return rsqrtf(sum / float(width) + eps);
}

// The body is a device function shared by the kernel of its own and by the one-launch small step: the calling
// thread block (SK_THREADS threads) is number `block` of `n_blocks` working on the launch's units; `wait` is called
// once by every thread, after the weights of the first steps have been requested, and must return when the
// activations (the previous kernel's or phase's output) are visible.
template <int MT, int DB, bool F16, bool FOLD, typename Wait>
__device__ __forceinline__ void gemm_skinny_body(const SkinnyParams& p, uint8_t* sk_smem, int block, int n_blocks, Wait wait) {
  constexpr int STAGE_BYTES = (NT + 2 * MT) * 512;          // per warp and K step: 4 weight tiles, 2 MT row groups
  constexpr int RING_BYTES = DB * STAGE_BYTES;              // per warp
  constexpr int PART_FLOATS = MT * 16 * PART_STRIDE;        // per warp
  // The partial tiles of the reduction get their own shared memory when it fits; else they reuse the rings.
  constexpr bool ALIAS = SK_WARPS * (RING_BYTES + PART_FLOATS * 4) > 227 * 1024;
  static_assert(!ALIAS || PART_FLOATS * 4 <= RING_BYTES, "a warp's partial tile must fit its own ring");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const uint32_t ring = smem_u32(sk_smem) + warp * RING_BYTES + lane * 16;
  float* part_all = reinterpret_cast<float*>(sk_smem + (ALIAS ? 0 : SK_WARPS * RING_BYTES));
  constexpr int PART_PITCH = ALIAS ? RING_BYTES / 4 : PART_FLOATS;   // floats between two warps' partial tiles
  float* part = part_all + warp * PART_PITCH;

  const int units = p.mode == kGemmGateUp ? p.N >> 4 : p.N >> 5;
  // 32-wide K steps, dealt to the warps in turn: warp w takes steps w, w + 8, ...  The eight warps move through
  // the K range together, so at any moment the block reads 512 contiguous bytes of each weight row -- a run long
  // enough for the DRAM pages it opens.  (Contiguous per-warp K slices would make 8 x 32 separate 64-byte streams.)
  const int steps = p.K >> 5;
  const int n = (steps - warp + SK_WARPS - 1) / SK_WARPS;
  const size_t k_off = (size_t(warp) * 32 + t * 8) * 2;     // byte offset of this lane's first 16 bytes in a row
  constexpr int STEP_BYTES = SK_WARPS * 64;                 // from one of the warp's steps to its next

  const uint8_t* wrow[NT];
  auto set_rows = [&](int unit) {
#pragma unroll
    for (int j = 0; j < NT; ++j) wrow[j] = unit_row(p, unit, j, g) + k_off;
  };
  // activation rows of this lane: rows 16 i + g and 16 i + g + 8 (clamped into the step)
  const uint8_t* arow[MT][2];
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      int r = 16 * i + 8 * h + g;
      r = r < p.T ? r : p.T - 1;
      arow[i][h] = static_cast<const uint8_t*>(p.a) + size_t(r) * p.K * 2 + k_off;
    }
  auto issue_b = [&](int s, int slot) {                     // weights of step s of this warp's slice
#pragma unroll
    for (int j = 0; j < NT; ++j) cp_async16(ring + slot * STAGE_BYTES + j * 512, wrow[j] + size_t(s) * STEP_BYTES);
  };
  auto issue_a = [&](int s, int slot) {                     // activations of the same step
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
      for (int h = 0; h < 2; ++h)
        cp_async16(ring + slot * STAGE_BYTES + (NT + 2 * i + h) * 512, arow[i][h] + size_t(s) * STEP_BYTES);
  };
  auto prologue = [&]() {
#pragma unroll
    for (int s = 0; s < DB - 1; ++s) {
      if (s < n) {
        issue_b(s, s);
        issue_a(s, s);
      }
      cp_async_commit();
    }
  };

  int unit = block;
  if (unit < units) {                                       // weights never change: fetch them before the wait
    set_rows(unit);
#pragma unroll
    for (int s = 0; s < DB - 1; ++s)
      if (s < n) issue_b(s, s);
  }
  // the epilogue row of this thread and what it needs from the step's metadata (written before the step's first kernel)
  const int e_row = threadIdx.x >> 2, e_jq = (threadIdx.x & 3) * 4;
  const bool e_ok = e_row < MT * 16 && e_row < p.T;
  int e_pos = 0, e_slot = 0;
  if (p.mode == kGemmQkv && e_ok) {
    e_pos = p.tok_pos[e_row];
    e_slot = p.tok_slot[e_row];
  }
  wait();
  if (unit < units) {
#pragma unroll
    for (int s = 0; s < DB - 1; ++s) {
      if (s < n) issue_a(s, s);
      cp_async_commit();
    }
  }
  // folded RMSNorm, consuming side: r of this thread's epilogue row, on its way while the first unit streams
  float rs_in = 1.f;
  if (FOLD && p.in_row_rs != nullptr && int(threadIdx.x >> 2) < p.T) rs_in = __ldcg(p.in_row_rs + (threadIdx.x >> 2));
  if (FOLD && p.in_row_ss != nullptr) rs_in = row_norm_factor(p.in_row_ss, p.K >> 5, p.K >> 5, int(threadIdx.x >> 2), p.T, p.K, p.norm_eps);
  int* last_unit = reinterpret_cast<int*>(part_all + SK_WARPS * PART_PITCH);   // FOLD: one word behind the partial tiles

  for (; unit < units; unit += n_blocks) {
    // What the epilogue will read from memory is requested now, so that it has arrived when the K loop ends: the
    // output block to add to, the gains of a folded norm, the rotation of the row's position.
    float4 y_pre_lo = make_float4(0.f, 0.f, 0.f, 0.f), y_pre_hi = y_pre_lo, cs0 = y_pre_lo, cs1 = y_pre_lo;
    uint2 ng_lo = make_uint2(0u, 0u), ng_hi = ng_lo;
    if (e_ok) {
      if (p.mode == kGemmResid) {
        if (p.accumulate) {
          const float4* y_lo = reinterpret_cast<const float4*>(p.y + size_t(e_row) * p.N + unit * 32 + e_jq);
          y_pre_lo = __ldcg(y_lo);                           // (through the L2: see the one-launch small step)
          y_pre_hi = __ldcg(y_lo + 4);
        }
        if (FOLD && p.norm_gain != nullptr) {
          ng_lo = __ldg(reinterpret_cast<const uint2*>(p.norm_gain + unit * 32 + e_jq));
          ng_hi = __ldg(reinterpret_cast<const uint2*>(p.norm_gain + unit * 32 + e_jq + 16));
        }
      } else if (p.mode == kGemmQkv) {
        const int upr = p.head_dim >> 5, head = unit / upr, sub = unit - head * upr;
        if (head < p.q_dim / p.head_dim + p.n_kv_heads) {
          const float4* cs = reinterpret_cast<const float4*>(p.rope + size_t(e_pos) * (p.head_dim >> 1) + sub * 16 + e_jq);
          cs0 = cs[0];
          cs1 = cs[1];
        }
      }
    }
    float acc[MT][NT][4];
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
      for (int j = 0; j < NT; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

    int slot = 0, fill = DB - 1;                            // ring slot of step s / of step s + DB - 1
    for (int s = 0; s < n; ++s) {
      if (s + DB - 1 < n) {
        issue_b(s + DB - 1, fill);
        issue_a(s + DB - 1, fill);
      }
      cp_async_commit();
      cp_async_wait<DB - 1>();
      const uint32_t at = ring + slot * STAGE_BYTES;
      uint4 b[NT];
#pragma unroll
      for (int j = 0; j < NT; ++j) b[j] = lds16(at + j * 512);
#pragma unroll
      for (int i = 0; i < MT; ++i) {
        const uint4 lo = lds16(at + (NT + 2 * i) * 512), hi = lds16(at + (NT + 2 * i + 1) * 512);
        // the two MMAs on one accumulator are kept apart: four independent ones run between them
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_16816<F16>(acc[i][j], lo.x, hi.x, lo.y, hi.y, b[j].x, b[j].y);
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_16816<F16>(acc[i][j], lo.z, hi.z, lo.w, hi.w, b[j].z, b[j].w);
      }
      slot = slot + 1 == DB ? 0 : slot + 1;
      fill = fill + 1 == DB ? 0 : fill + 1;
    }
    cp_async_wait<0>();

    // the next unit's first steps travel while this one is reduced and written (when the rings stay free)
    const int next = unit + n_blocks;
    if (!ALIAS && next < units) {
      set_rows(next);
      prologue();
    }

    // partial tiles -> shared memory
#pragma unroll
    for (int i = 0; i < MT; ++i)
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        float* at = part + (16 * i + g) * PART_STRIDE + 8 * j + 2 * t;
        *reinterpret_cast<float2*>(at) = make_float2(acc[i][j][0], acc[i][j][1]);
        *reinterpret_cast<float2*>(at + 8 * PART_STRIDE) = make_float2(acc[i][j][2], acc[i][j][3]);
      }
    __syncthreads();

    // sum of the 8 warps' partials in warp order, then the epilogue of the mode.  Thread -> row tid / 4 and the
    // tile columns jq .. jq + 3 ("lo") and 16 + jq .. 16 + jq + 3 ("hi").
    const int row = threadIdx.x >> 2, jq = (threadIdx.x & 3) * 4;
    if (row < MT * 16 && row < p.T) {
      const float* src = part_all + row * PART_STRIDE + jq;
      float4 lo = *reinterpret_cast<const float4*>(src), hi = *reinterpret_cast<const float4*>(src + 16);
#pragma unroll
      for (int w = 1; w < SK_WARPS; ++w) {
        const float4 l = *reinterpret_cast<const float4*>(src + w * PART_PITCH);
        const float4 h = *reinterpret_cast<const float4*>(src + w * PART_PITCH + 16);
        lo.x += l.x; lo.y += l.y; lo.z += l.z; lo.w += l.w;
        hi.x += h.x; hi.y += h.y; hi.z += h.z; hi.w += h.w;
      }
      if (FOLD && (p.in_row_rs != nullptr || p.in_row_ss != nullptr)) {
        lo.x *= rs_in; lo.y *= rs_in; lo.z *= rs_in; lo.w *= rs_in;
        hi.x *= rs_in; hi.y *= rs_in; hi.z *= rs_in; hi.w *= rs_in;
      }
      if (p.mode == kGemmResid) {
        float4* y_lo = reinterpret_cast<float4*>(p.y + size_t(row) * p.N + unit * 32 + jq);
        float4* y_hi = y_lo + 4;
        if (p.gate_mod) {                                    // conditioned block: gate vector of the row's sequence
          const float4* gate = reinterpret_cast<const float4*>(p.gate_mod + (size_t(p.tok_seq[row]) * 6 + p.gate_which) * p.N +
                                                               unit * 32 + jq);
          const float4 g_lo = __ldg(gate), g_hi = __ldg(gate + 4);
          lo.x *= g_lo.x; lo.y *= g_lo.y; lo.z *= g_lo.z; lo.w *= g_lo.w;
          hi.x *= g_hi.x; hi.y *= g_hi.y; hi.z *= g_hi.z; hi.w *= g_hi.w;
        }
        if (p.accumulate) {
          const float4 a = y_pre_lo, b = y_pre_hi;
          lo.x += a.x; lo.y += a.y; lo.z += a.z; lo.w += a.w;
          hi.x += b.x; hi.y += b.y; hi.z += b.z; hi.w += b.w;
        }
        *y_lo = lo;
        *y_hi = hi;
        if (FOLD && p.norm_gain != nullptr) {
          // folded RMSNorm, producing side: the next GEMM's operand and this unit's share of the row's sum of squares
          // (the four threads of a row are neighbours in a warp)
          const uint2 g_lo = ng_lo, g_hi = ng_hi;
          float v[8] = {lo.x * __uint_as_float(g_lo.x << 16), lo.y * __uint_as_float(g_lo.x & 0xffff0000u),
                        lo.z * __uint_as_float(g_lo.y << 16), lo.w * __uint_as_float(g_lo.y & 0xffff0000u),
                        hi.x * __uint_as_float(g_hi.x << 16), hi.y * __uint_as_float(g_hi.x & 0xffff0000u),
                        hi.z * __uint_as_float(g_hi.y << 16), hi.w * __uint_as_float(g_hi.y & 0xffff0000u)};
          if (p.norm_h_f16 && p.status) note_f16_saturation(v, p.status);
          __nv_bfloat16* hrow = p.norm_h + size_t(row) * p.N + unit * 32 + jq;
          *reinterpret_cast<uint2*>(hrow) = make_uint2(pack_act(v[0], v[1], p.norm_h_f16 != 0), pack_act(v[2], v[3], p.norm_h_f16 != 0));
          *reinterpret_cast<uint2*>(hrow + 16) = make_uint2(pack_act(v[4], v[5], p.norm_h_f16 != 0), pack_act(v[6], v[7], p.norm_h_f16 != 0));
          float ss = lo.x * lo.x + lo.y * lo.y + lo.z * lo.z + lo.w * lo.w + hi.x * hi.x + hi.y * hi.y + hi.z * hi.z + hi.w * hi.w;
          ss += __shfl_xor_sync(0xfu << (lane & 28), ss, 1);
          ss += __shfl_xor_sync(0xfu << (lane & 28), ss, 2);
          if ((threadIdx.x & 3) == 0) p.row_ss[size_t(row) * p.ss_stride + unit] = ss;
        }
      } else if (p.mode == kGemmGateUp) {
        const float gt[4] = {lo.x, lo.y, lo.z, lo.w}, up[4] = {hi.x, hi.y, hi.z, hi.w};
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = __fdividef(gt[e] * up[e], 1.f + __expf(-gt[e]));   // silu(gate) * up
        if (p.act_f16 && p.status) note_f16_saturation(v, p.status);
        uint2 out;
        out.x = pack_act(v[0], v[1], p.act_f16 != 0);
        out.y = pack_act(v[2], v[3], p.act_f16 != 0);
        *reinterpret_cast<uint2*>(p.act + size_t(row) * p.N + unit * 16 + jq) = out;
      } else {
        const int Dh = p.head_dim, half = Dh >> 1, upr = Dh >> 5;
        const int head = unit / upr, sub = unit - head * upr;
        const int i0 = sub * 16 + jq;                        // first rotation pair / first element inside the head
        const int n_q_heads = p.q_dim / Dh;
        float a[4] = {lo.x, lo.y, lo.z, lo.w}, b[4] = {hi.x, hi.y, hi.z, hi.w};
        const int region = head < n_q_heads ? 0 : head < n_q_heads + p.n_kv_heads ? 1 : 2;
        if (p.qkv_bias[region]) {                            // the bias comes before the rotation
          const int col = (head - (region == 0 ? 0 : region == 1 ? n_q_heads : n_q_heads + p.n_kv_heads)) * Dh + i0;
          const uint2 wl = __ldg(reinterpret_cast<const uint2*>(p.qkv_bias[region] + col));
          const uint2 wh = __ldg(reinterpret_cast<const uint2*>(p.qkv_bias[region] + col + half));
          a[0] += __uint_as_float(wl.x << 16); a[1] += __uint_as_float(wl.x & 0xffff0000u);
          a[2] += __uint_as_float(wl.y << 16); a[3] += __uint_as_float(wl.y & 0xffff0000u);
          b[0] += __uint_as_float(wh.x << 16); b[1] += __uint_as_float(wh.x & 0xffff0000u);
          b[2] += __uint_as_float(wh.y << 16); b[3] += __uint_as_float(wh.y & 0xffff0000u);
        }
        if (head < n_q_heads + p.n_kv_heads) {               // q and k heads are rotated
          const float4 t0 = cs0, t1 = cs1;                   // (cos, sin) of pairs i0 .. i0 + 3, requested at the unit's start
          const float c[4] = {t0.x, t0.z, t1.x, t1.z}, sn[4] = {t0.y, t0.w, t1.y, t1.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float x0 = a[e], x1 = b[e];
            a[e] = x0 * c[e] - x1 * sn[e];
            b[e] = x1 * c[e] + x0 * sn[e];
          }
        }
        uint2 o_lo, o_hi;
        o_lo.x = pack_act(a[0], a[1], false); o_lo.y = pack_act(a[2], a[3], false);
        o_hi.x = pack_act(b[0], b[1], false); o_hi.y = pack_act(b[2], b[3], false);
        __nv_bfloat16* dst;
        if (head < n_q_heads) {
          dst = p.q_out + size_t(row) * p.q_dim + head * Dh + i0;
        } else {
          const int hk = head - n_q_heads;
          const int slot = e_slot;
          dst = hk < p.n_kv_heads ? cache_row(p.k_cache, slot, hk, p.n_kv_heads, Dh) + i0
                                  : cache_row(p.v_cache, slot, hk - p.n_kv_heads, p.n_kv_heads, Dh) + i0;
        }
        *reinterpret_cast<uint2*>(dst) = o_lo;
        *reinterpret_cast<uint2*>(dst + half) = o_hi;
      }
    }
    __syncthreads();                                         // the partial tiles are free again
    if (FOLD && p.mode == kGemmResid && p.norm_gain != nullptr && p.units_done != nullptr) {
      // the block that delivers the last unit turns the partial sums into every row's r (for a tiled GEMM behind the
      // norm).  (The barrier above orders the block's stores before thread 0's fence.)
      if (threadIdx.x == 0) {
        __threadfence();
        *last_unit = atomicAdd(p.units_done, 1) == units - 1;
      }
      __syncthreads();
      if (*last_unit) {
        __threadfence();
        const float r = row_norm_factor(p.row_ss, p.ss_stride, units, row, p.T, p.N, p.norm_eps);
        if ((threadIdx.x & 3) == 0 && row < p.T) p.row_rs[row] = r;
        if (threadIdx.x == 0) *p.units_done = 0;             // ready for the next launch
      }
    }
    if (ALIAS && next < units) {
      set_rows(next);
      prologue();
    }
  }
}

template <int MT, int DB, bool F16, bool FOLD>
__global__ void __launch_bounds__(SK_THREADS, 1) gemm_skinny_kernel(const SkinnyParams p) {
  extern __shared__ __align__(16) uint8_t sk_smem[];
  log_smid(p.smid_log);
  gemm_skinny_body<MT, DB, F16, FOLD>(p, sk_smem, int(blockIdx.x), int(gridDim.x), [] {
    griddep_wait();
    griddep_launch_dependents();
  });
}

template <int MT, int DB>
constexpr int skinny_smem() {
  constexpr int rings = SK_WARPS * DB * (NT + 2 * MT) * 512, both = rings + SK_WARPS * MT * 16 * PART_STRIDE * 4;
  return (both > 227 * 1024 ? rings : both) + 16;            // + the word of the folded norm's last-unit flag
}
constexpr int DB1 = 8, DB2 = 6, DB4 = 4;                     // ring depths by row-tile count
static_assert(skinny_smem<1, DB1>() <= 227 * 1024 && skinny_smem<2, DB2>() <= 227 * 1024 && skinny_smem<4, DB4>() <= 227 * 1024,
              "rings and partial tiles must fit one SM");

template <int MT, int DB>
cudaError_t launch_one(const SkinnyParams& p, int grid, cudaStream_t stream) {
  constexpr int smem = skinny_smem<MT, DB>() < kMinSmemBytes ? kMinSmemBytes : skinny_smem<MT, DB>();
  const bool fold = p.norm_gain != nullptr || p.in_row_rs != nullptr || p.in_row_ss != nullptr;
  if (p.ab_f16) {
    if (fold) return launch_step_kernel(gemm_skinny_kernel<MT, DB, true, true>, grid, SK_THREADS, smem, stream, p.overlap != 0, p);
    return launch_step_kernel(gemm_skinny_kernel<MT, DB, true, false>, grid, SK_THREADS, smem, stream, p.overlap != 0, p);
  }
  if (fold) return launch_step_kernel(gemm_skinny_kernel<MT, DB, false, true>, grid, SK_THREADS, smem, stream, p.overlap != 0, p);
  return launch_step_kernel(gemm_skinny_kernel<MT, DB, false, false>, grid, SK_THREADS, smem, stream, p.overlap != 0, p);
}
template <int MT, int DB>
cudaError_t set_one() {
  constexpr int smem = skinny_smem<MT, DB>() < kMinSmemBytes ? kMinSmemBytes : skinny_smem<MT, DB>();
  cudaError_t e = set_kernel_smem(gemm_skinny_kernel<MT, DB, true, false>, smem);
  if (e == cudaSuccess) e = set_kernel_smem(gemm_skinny_kernel<MT, DB, false, false>, smem);
  if (e == cudaSuccess) e = set_kernel_smem(gemm_skinny_kernel<MT, DB, true, true>, smem);
  if (e == cudaSuccess) e = set_kernel_smem(gemm_skinny_kernel<MT, DB, false, true>, smem);
  return e;
}


// ============================================================ one-launch small step ==
// Shared memory: the weight-streaming GEMM's rings and partial tiles from offset 0 (the decode attention's page rings
// use the front of the same area in their phase), the decode attention's mbarriers behind them.
constexpr int SS_BAR_OFFSET = (skinny_smem<1, DB1>() + 1023) / 1024 * 1024;
constexpr int SS_SMEM = SS_BAR_OFFSET + 512 + 1024;          // + barriers + room to align the base
static_assert(SS_SMEM <= 227 * 1024 && SS_SMEM >= kMinSmemBytes, "one block per SM");
static_assert(DC_WARPS * DC_STAGES * 2 * Geom<128>::PAGE_BYTES <= SS_BAR_OFFSET, "the page rings fit in front of the barriers");
static_assert(DC_WARPS * 32 <= SK_THREADS, "the decode phase uses the first warps of the block");

// Arrives at the grid barrier and waits until `target` blocks have (bounded: gives up after the wait limit, records
// HS_ERR_TIMEOUT and returns false in every thread of the block).
__device__ __forceinline__ bool grid_barrier(int* counter, int target, int* status) {
  __syncthreads();                      // this block's writes of the phase come before thread 0's fence
  int failed = 0;
  if (threadIdx.x == 0) {
    // release: the block's writes (ordered before this thread by the barrier above) are visible to whoever sees the count
    asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(counter) : "memory");
    const unsigned long long t0 = globaltimer_ns();
    for (;;) {
      int seen;
      asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
      if (seen >= target) break;
      if (globaltimer_ns() - t0 > kWaitLimitNs) {
        atomicExch(status, kErrTimeout);
        failed = 1;
        break;
      }
      __nanosleep(32);
    }
  }
  return __syncthreads_or(failed) == 0;   // the acquire above, then this barrier: every thread sees the other blocks' writes
}

template <int DH, bool F16>
__global__ void __launch_bounds__(SK_THREADS, 1) small_step_kernel(const __grid_constant__ SmallStepParams p) {
  extern __shared__ uint8_t ss_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(ss_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* dc_bars = reinterpret_cast<uint64_t*>(smem + SS_BAR_OFFSET);
  log_smid(p.smid_log);
  const int block = int(blockIdx.x), grid = int(gridDim.x);
  const int qkv_n = p.q_dim + 2 * p.kv_dim;
  const int nb_qkv = min(grid, qkv_n >> 5), nb_attn = min(grid, p.attn.decode_group ? p.attn.n_decode_items / DC_WARPS : p.attn.n_decode_items), nb_d = min(grid, p.d >> 5),
            nb_gu = min(grid, p.F >> 4);
  int arrived = 0;                      // grid barriers this block has been through
  bool dead = false;                    // a barrier ran out of time: no further waits, leave after the phase
  auto barrier = [&] {
    ++arrived;
    if (!dead && !grid_barrier(p.grid_bar, arrived * grid, p.status)) dead = true;
  };
  auto base = [&](const void* a, int K, int N, int mode) {
    SkinnyParams k{};
    k.a = a; k.T = p.T; k.K = K; k.N = N; k.mode = mode;
    k.ab_f16 = F16 ? 1 : 0;
    k.status = p.status;
    return k;
  };
  auto fold_out = [&](SkinnyParams& k, const __nv_bfloat16* gain) {
    k.norm_gain = gain; k.norm_h = p.h; k.norm_h_f16 = F16 ? 1 : 0;
    k.row_ss = p.row_ss; k.ss_stride = p.d >> 5; k.norm_eps = p.eps;     // the consuming GEMM adds the partials itself
  };
  for (int l = 0; l < p.n_layers && !dead; ++l) {
    const SmallLayer L = p.layers[l];
    {  // QKV projection + RoPE + cache write (the norm in front of it: the step's first norm kernel, or folded)
      SkinnyParams k = base(p.h, p.d, qkv_n, kGemmQkv);
      k.w[0] = L.w_q; k.w[1] = L.w_k; k.w[2] = L.w_v;
      k.q_dim = p.q_dim; k.kv_dim = p.kv_dim; k.head_dim = p.head_dim; k.n_kv_heads = p.n_kv_heads;
      k.q_out = p.q;
      k.k_cache = p.kv_pool + (size_t(l) * 2 + 0) * p.layer_kv_elems;
      k.v_cache = p.kv_pool + (size_t(l) * 2 + 1) * p.layer_kv_elems;
      k.tok_pos = p.tok_pos; k.tok_slot = p.tok_slot; k.rope = p.rope;
      for (int i = 0; i < 3; ++i) k.qkv_bias[i] = L.bias[i];
      if (l > 0) { k.in_row_ss = p.row_ss; k.norm_eps = p.eps; }
      auto w = [&] { if (l > 0) barrier(); };
      if (block < nb_qkv) gemm_skinny_body<1, DB1, F16, true>(k, smem, block, nb_qkv, w);
      else w();
    }
    if (dead) break;
    {  // decode attention
      auto w = [&] { barrier(); };
      if (block < nb_attn) {
        attn_decode_body<DH>(p.attn, l, p.counters + 2 * l, smem, dc_bars, block, nb_attn, w);
        if (threadIdx.x == 0)           // the barriers' memory belongs to the next phase's rings no more, but end their life
          for (int i = 0; i < DC_WARPS * DC_STAGES; ++i) mbar_inval(&dc_bars[i]);
        __syncthreads();
      } else {
        w();
      }
    }
    if (dead) break;
    {  // out-projection + residual add (+ the MLP norm's operand, sums and r)
      SkinnyParams k = base(p.o, p.q_dim, p.d, kGemmResid);
      k.w[0] = L.w_o; k.y = p.x; k.accumulate = 1;
      fold_out(k, L.g_mlp);
      auto w = [&] { barrier(); };
      if (block < nb_d) gemm_skinny_body<1, DB1, F16, true>(k, smem, block, nb_d, w);
      else w();
    }
    if (dead) break;
    {  // gate / up projection + SwiGLU
      SkinnyParams k = base(p.h, p.d, p.F, kGemmGateUp);
      k.w[0] = L.w_gate; k.w[1] = L.w_up;
      k.act = p.act; k.act_f16 = F16 ? 1 : 0;
      k.in_row_ss = p.row_ss; k.norm_eps = p.eps;
      auto w = [&] { barrier(); };
      if (block < nb_gu) gemm_skinny_body<1, DB1, F16, true>(k, smem, block, nb_gu, w);
      else w();
    }
    if (dead) break;
    {  // down-projection + residual add (+ the next layer's attention norm)
      SkinnyParams k = base(p.act, p.F, p.d, kGemmResid);
      k.w[0] = L.w_down; k.y = p.x; k.accumulate = 1;
      if (l + 1 < p.n_layers) fold_out(k, p.layers[l + 1].g_attn);
      auto w = [&] { barrier(); };
      if (block < nb_d) gemm_skinny_body<1, DB1, F16, true>(k, smem, block, nb_d, w);
      else w();
    }
  }
}

template <int DH, bool F16>
cudaError_t launch_small_one(const SmallStepParams& p, int grid, cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(grid), 1, 1);
  cfg.blockDim = dim3(SK_THREADS, 1, 1);
  cfg.dynamicSmemBytes = SS_SMEM;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;      // all blocks resident at once: they wait on one another
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, small_step_kernel<DH, F16>, p);
}

}  // namespace

bool gemm_skinny_supports(int T, int K, int N, int mode, int head_dim) {
  if (T < 1 || T > 64 || K < 32 || K % 32 != 0) return false;
  if (mode == kGemmResid) return N % 32 == 0;
  if (mode == kGemmGateUp) return N % 16 == 0;
  return head_dim % 32 == 0 && N % head_dim == 0;
}

// Which kernel is faster for this shape, from measurements on B200 (config-3 and talker dimensions, 8 .. 64 rows).
// A block of this kernel takes in about 70 KB/us and reads, per unit, 32 weight rows plus all (16 MT) activation
// rows of width K, with about 1.5 us per unit for set-up, reduction and epilogue; units run in rounds of one per SM.
// The tiled kernel streams a 64-wide K block in about 0.36 us (0.8 us with two weight boxes per stage, gate/up)
// and pays 3.5 us per link of a K-split chain.  So this kernel wins where the tiled one has too few tiles to
// occupy the device or needs a long chain (QKV, out-projection, down at few rows), and loses where there are
// tiles enough (gate/up of a wide FFN), because here every 32 columns re-read the activations.
// Depends on the shape and the device only, never on the SM budget: the two kernels round differently, and a
// step's result must not depend on its budget.  Rounds and waves are counted for the whole device.  Measured
// against the alternatives over budgets 148 / 111 / 74 at config-3 dimensions (ms per 28-layer decode-only step,
// all projections tiled -> this rule): 16 rows 4.39 -> 3.49, 5.42 -> 5.14, 5.74 -> 5.27; 32 rows 4.91 -> 4.36,
// 5.99 -> 5.80, 6.34 -> 6.15; 64 rows 5.72 -> 5.38, 7.21 -> 7.43, 8.06 -> 8.32 (with its unit count just below
// the SM count this kernel needs a second round as soon as the budget drops, which at 64 rows costs 3 %).
bool gemm_skinny_wins(int T, int K, int N, int mode, int head_dim, int sm_count) {
  if (!gemm_skinny_supports(T, K, N, mode, head_dim)) return false;
  const int mt = T <= 16 ? 1 : T <= 32 ? 2 : 4;
  const int units = mode == kGemmGateUp ? N / 16 : N / 32;
  const int rounds = (units + sm_count - 1) / sm_count;
  const double mine = rounds * (1.5 + double(32 + 16 * mt) * K * 2 / 70e3);
  const int k_blocks = (K + 63) / 64;
  double tiled;
  if (mode == kGemmResid) {
    const int bn = gemm_pick_bn(T, N, sm_count), ks = gemm_pick_ksplit(T, N, K, bn, sm_count);
    const int tiles = (N + bn - 1) / bn, waves = (tiles * ks + sm_count - 1) / sm_count;
    tiled = gemm_ksplit_cost_us(k_blocks, ks, waves);
  } else {
    const int tiles = (N + 127) / 128, waves = (tiles + sm_count - 1) / sm_count;
    tiled = double(waves) * k_blocks * (mode == kGemmGateUp ? 0.8 : 0.36);
  }
  return mine < tiled;
}

cudaError_t gemm_skinny_set_attributes() {
  cudaError_t e = set_one<1, DB1>();
  if (e == cudaSuccess) e = set_one<2, DB2>();
  if (e == cudaSuccess) e = set_one<4, DB4>();
  return e;
}

cudaError_t small_step_set_attributes() {
  cudaError_t e = set_kernel_smem(small_step_kernel<64, true>, SS_SMEM);
  if (e == cudaSuccess) e = set_kernel_smem(small_step_kernel<64, false>, SS_SMEM);
  if (e == cudaSuccess) e = set_kernel_smem(small_step_kernel<128, true>, SS_SMEM);
  if (e == cudaSuccess) e = set_kernel_smem(small_step_kernel<128, false>, SS_SMEM);
  return e;
}

cudaError_t launch_small_step(const SmallStepParams& p, int sm_budget, cudaStream_t stream) {
  if (p.T <= 0 || p.T > 16 || p.attn.n_decode_items <= 0) return cudaErrorInvalidValue;
  const int attn_work = p.attn.decode_group ? p.attn.n_decode_items / DC_WARPS : p.attn.n_decode_items;
  const int widest = std::max(std::max((p.q_dim + 2 * p.kv_dim) >> 5, attn_work), std::max(p.d >> 5, p.F >> 4));
  const int grid = widest < sm_budget ? widest : sm_budget;
  if (p.head_dim == 128) return p.f16 ? launch_small_one<128, true>(p, grid, stream) : launch_small_one<128, false>(p, grid, stream);
  return p.f16 ? launch_small_one<64, true>(p, grid, stream) : launch_small_one<64, false>(p, grid, stream);
}

cudaError_t launch_gemm_skinny(const SkinnyParams& p, int sm_budget, cudaStream_t stream) {
  if (p.T <= 0) return cudaSuccess;
  const int units = p.mode == kGemmGateUp ? p.N / 16 : p.N / 32;
  const int grid = units < sm_budget ? units : sm_budget;
  if (p.T <= 16) return launch_one<1, DB1>(p, grid, stream);
  if (p.T <= 32) return launch_one<2, DB2>(p, grid, stream);
  return launch_one<4, DB4>(p, grid, stream);
}

}  // namespace hs
