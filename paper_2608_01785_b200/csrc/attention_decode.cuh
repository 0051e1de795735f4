// Decode-side causal GQA attention over the paged bf16 KV cache: TMA-staged K/V pages, warp-level
// tensor-core tiles (mma.sync m16n8k16) and an fp32 online softmax in the log2 domain.  (The prefill
// kernel lives in attention_prefill.cu.)
//
//   decode kernel    work item = (sequence, KV head, run of at most 512 keys); rows = the G query heads of the
//                    single new token.  Eight autonomous warps per block, each streaming its own item's
//                    pages through a private TMA ring and writing one partial (max, sum, output) per
//                    item.  HBM-bound: 8 warps x 2 (K page, V page) pairs x 8 KB in flight per SM.
//                    The warp that finishes the last split of a (sequence, KV head) merges that group's
//                    partials in split order (a group with a single split writes its output directly).
// Work items are listed on the host independently of the SM budget and handed out through an atomic
// queue head; an item's result does not depend on which block ran it, and every reduction has a fixed
// order, so outputs are bit-identical across budgets.
//
// A page block [16 keys][Dh] arrives as Dh/64 tiles of [16][64] with the 128-byte swizzle, which makes
// every ldmatrix below bank-conflict free.  Keys past the end of a sequence (the unused tail of its last
// page, or pages of a ragged last block that were never fetched) may hold arbitrary bytes: scores are
// masked by selection and the matching V fragments are zeroed, so they cannot reach the output.
#pragma once
#include <math.h>

#include "kernels.h"
#include "ptx.cuh"

namespace hs {
namespace {

constexpr float kLog2e = 1.4426950408889634f;

template <int DH>
struct Geom {
  static constexpr int HALVES = DH / 64;
  static constexpr int PAGE_BYTES = HALVES * 2048;   // [HALVES][16 keys][128 B]
  static constexpr int CHUNKS = DH / 8;              // 16-byte chunks per row
};

// Byte offset of (key kk, 16-byte chunk cc) inside a page block.
__device__ __forceinline__ int kv_off(int kk, int cc) {
  return (cc >> 3) * 2048 + kk * 128 + (((cc & 7) ^ (kk & 7)) << 4);
}
// First pool row (unit: one key's Dh elements of one KV head) of (layer, K|V, page, head).
__device__ __forceinline__ int pool_row(const AttnParams& p, int layer, int kv, int page, int hk) {
  return (((layer * 2 + kv) * p.num_pages + page) * p.n_kv_heads + hk) * 16;
}
template <int DH>
__device__ __forceinline__ void load_page(const AttnParams& p, int layer, uint8_t* dst, uint64_t* bar, int kv, int page, int hk) {
  const int row = pool_row(p, layer, kv, page, hk);
#pragma unroll
  for (int h = 0; h < Geom<DH>::HALVES; ++h) tma_load_2d(dst + h * 2048, &p.tm_kv, bar, h * 64, row);
}
__device__ __forceinline__ float quad_max(float v) {
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
  return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_sum(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  return v + __shfl_xor_sync(0xffffffffu, v, 2);
}
// Zeroes the halves of a V fragment register whose keys (k, k + 1) are not below n_valid.
__device__ __forceinline__ uint32_t mask_v(uint32_t r, int k, int n_valid) {
  if (k >= n_valid) return 0u;
  if (k + 1 >= n_valid) return r & 0x0000ffffu;
  return r;
}

// Merges the partials of one (sequence, KV head) group -- items first .. first + splits - 1 -- in split
// order and writes the normalised output rows.  LPH lanes share one query head, each owning DH / LPH
// contiguous columns.  A lone warp does this at the tail of the kernel, so what counts is latency: the
// partial outputs travel by asynchronous copies into the warp's own (now idle) page ring, used as two
// halves of PS splits each -- while one half is folded into the running sum the other is in flight -- laid
// out [split][float4 index][lane] so that every lane reads back only what it copied itself, conflict-free.
// The running maximum is updated per half (online rescaling); the order of all operations is fixed.
template <int DH, int LPH, int RING_BYTES>
__device__ __forceinline__ void merge_group(const float* part_o, const float* part_ml, uint8_t* ring, int first,
                                            int splits, int G, int lane, __nv_bfloat16* orow, bool f16, int* status) {
  constexpr int NV = DH / 4 / LPH;                 // float4 per lane and split
  constexpr int PS = RING_BYTES / 2 / (NV * 512) < 4 ? RING_BYTES / 2 / (NV * 512) : 4;   // splits per half
  static_assert(PS >= 1, "half a ring holds one split");
  const int g = lane / LPH, part = lane % LPH;
  if (g < G) {
    const float2* ml_g = reinterpret_cast<const float2*>(part_ml) + size_t(first) * 16 + g;   // + j * 16
    const uint32_t ring_u32 = smem_u32(ring) + lane * 16;
    const float4* ring_f4 = reinterpret_cast<const float4*>(ring) + lane;
    float2 mlv[2][PS];
    auto request = [&](int j0, int half) {         // splits j0 .. j0 + PS - 1 into one half of the ring
#pragma unroll
      for (int u = 0; u < PS; ++u) {
        if (j0 + u < splits) {
          const float4* src = reinterpret_cast<const float4*>(part_o + (size_t(first + j0 + u) * 16 + g) * DH) + part * NV;
#pragma unroll
          for (int i = 0; i < NV; ++i)
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(ring_u32 + ((half * PS + u) * NV + i) * 512),
                         "l"(src + i)
                         : "memory");
          mlv[half][u] = __ldcg(&ml_g[size_t(j0 + u) * 16]);
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    float mm = -INFINITY, ll = 0.f;
    float4 acc[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) acc[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    request(0, 0);
    request(PS, 1);
    int half = 0;
    for (int j0 = 0; j0 < splits; j0 += PS, half ^= 1) {
      asm volatile("cp.async.wait_group 1;" ::: "memory");     // the older of the two halves has landed
      float pm = mm;
      if (half == 0) {
#pragma unroll
        for (int u = 0; u < PS; ++u) if (j0 + u < splits) pm = fmaxf(pm, mlv[0][u].x);
      } else {
#pragma unroll
        for (int u = 0; u < PS; ++u) if (j0 + u < splits) pm = fmaxf(pm, mlv[1][u].x);
      }
      const float sc = exp2f(mm - pm);                         // 0 on the first half (mm = -inf)
      mm = pm;
      ll *= sc;
#pragma unroll
      for (int i = 0; i < NV; ++i) { acc[i].x *= sc; acc[i].y *= sc; acc[i].z *= sc; acc[i].w *= sc; }
#pragma unroll
      for (int u = 0; u < PS; ++u) {
        if (j0 + u < splits) {
          const float2 ml = half == 0 ? mlv[0][u] : mlv[1][u];
          const float f = exp2f(ml.x - mm);
          ll += f * ml.y;
#pragma unroll
          for (int i = 0; i < NV; ++i) {
            const float4 v = ring_f4[((half * PS + u) * NV + i) * 32];
            acc[i].x += f * v.x; acc[i].y += f * v.y; acc[i].z += f * v.z; acc[i].w += f * v.w;
          }
        }
      }
      if (half == 0) request(j0 + 2 * PS, 0);                  // refill the half just read (may be empty)
      else request(j0 + 2 * PS, 1);
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    const float inv = 1.f / ll;
    if (f16) {
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const float v4[4] = {acc[i].x, acc[i].y, acc[i].z, acc[i].w};
        note_f16_saturation(v4, status, inv);
      }
    }
    __nv_bfloat16* dst = orow + g * DH + part * NV * 4;
#pragma unroll
    for (int i = 0; i < NV; ++i)
      *reinterpret_cast<uint2*>(dst + 4 * i) =
          make_uint2(pack_act(acc[i].x * inv, acc[i].y * inv, f16), pack_act(acc[i].z * inv, acc[i].w * inv, f16));
  }
  // the ring goes back to the copy engine for the next item: order these generic-proxy accesses before it
  fence_proxy_async();
  __syncwarp();
}

// ==================================================================== decode ==
// Every warp is its own pipeline: it pulls a work item from the queue, streams the item's pages through
// a private ring of DC_STAGES (K page, V page) slots that its lane 0 fills by TMA a few pages ahead, and
// writes the item's partial (max, sum, output) straight from its registers.  There is no producer warp,
// no "slot free" barrier (a slot is refilled by the warp that has just finished reading it) and no
// block-level synchronisation after start-up, so an SM keeps DC_WARPS x (DC_STAGES - 1) pages in flight.
// Measured on B200 (warps x slots of 8 KB, the 192 KB an SM offers): 8 x 3 and 6 x 4 take the same time at the full
// budget (config-3 decode tick 5.17 / 5.15 ms), 8 x 3 is 5-8 % faster at 74 and 37 SMs, 4 x 6 is 9 % slower everywhere.
constexpr int DC_WARPS = kDecodeKernelWarps, DC_THREADS = DC_WARPS * 32, DC_STAGES = 3;

template <int DH>
constexpr int dc_smem_bytes() {
  int b = 1024 + DC_WARPS * DC_STAGES * 2 * Geom<DH>::PAGE_BYTES + 512;
  return b > kMinSmemBytes ? b : kMinSmemBytes;
}

// The body of the decode kernel as a device function, so that the kernel of its own and the one-launch small step
// share it.  `smem`: 1024-byte aligned, DC_WARPS * DC_STAGES * 2 pages; `full_all`: DC_WARPS * DC_STAGES mbarriers
// followed by one int (the abort flag) in shared memory outside that area.  The calling thread block is number
// `block` of `n_blocks` working on the launch's items; it may have more than DC_WARPS warps (the others only take
// part in the two block barriers).  `layer` and `counters` (this layer's two queue heads) stand in for the fields of
// the same names in `p`, which holds the tensor map and therefore cannot be copied per layer.  `wait` is called once by every thread, after the set-up and the requests that do
// not depend on the previous kernel or phase, and must return when that predecessor's writes are visible.
template <int DH, typename Wait>
__device__ __forceinline__ void attn_decode_body(const AttnParams& p, int layer, int32_t* counters, uint8_t* smem,
                                                 uint64_t* full_all, int block, int n_blocks, Wait wait) {
  using G_ = Geom<DH>;
  constexpr int SLOT_BYTES = 2 * G_::PAGE_BYTES;    // K page then V page
  volatile int* abort_flag = reinterpret_cast<volatile int*>(full_all + DC_WARPS * DC_STAGES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool worker = warp < DC_WARPS;
  const int G = p.n_q_heads / p.n_kv_heads;
  const int q_dim = p.n_q_heads * DH;
  const float scale_log2 = kLog2e / sqrtf(float(DH));

  if (threadIdx.x == 0) {
    for (int i = 0; i < DC_WARPS * DC_STAGES; ++i) mbar_init(&full_all[i], 1);
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&p.tm_kv);
  }
  __syncthreads();

  uint8_t* slots = smem + (worker ? warp : 0) * DC_STAGES * SLOT_BYTES;
  uint64_t* full = full_all + (worker ? warp : 0) * DC_STAGES;
  uint32_t issued = 0, consumed = 0;      // pages this warp has requested / finished, over all its items
  auto issue = [&](int page, int hk) {      // lane 0: request one page of an item
    const uint32_t st = issued % DC_STAGES;
    mbar_expect_tx(&full[st], SLOT_BYTES);
    load_page<DH>(p, layer, slots + st * SLOT_BYTES, &full[st], 0, page, hk);
    load_page<DH>(p, layer, slots + st * SLOT_BYTES + G_::PAGE_BYTES, &full[st], 1, page, hk);
    ++issued;
  };

  // A warp's first item is its own index in the grid (no round trip to the queue head before the first page request);
  // the queue hands out the items after those.  The first item's record, its page ids and those of its first pages
  // that lie wholly inside the cached context are fetched before the wait for the previous kernel: the step's
  // metadata was copied before any kernel of the step started, and this step writes K / V at positions >= ctx only.
  int item = worker ? block * DC_WARPS + warp : p.n_decode_items;
  int4 it = make_int4(0, 0, 0, 0), dr = it;
  int my_page = 0, ahead = 0;             // ahead: pages of the current item already requested
  if (item < p.n_decode_items) {
    it = reinterpret_cast<const int4*>(p.decode_items)[2 * item];
    dr = reinterpret_cast<const int4*>(p.decode_items)[2 * item + 1];
    const int n_pages = (it.w - it.z + 15) >> 4;
    my_page = lane < n_pages ? p.block_tables[size_t(dr.x) * p.max_pages_per_seq + (it.z >> 4) + lane] : 0;
    const int ctx = p.seq_ctx[dr.x];
#pragma unroll
    for (int pi = 0; pi < DC_STAGES - 1; ++pi) {
      const int page = __shfl_sync(0xffffffffu, my_page, pi);
      const bool stable = pi < n_pages && it.z + (pi + 1) * 16 <= ctx && ahead == pi;
      if (stable) {
        if (lane == 0) issue(page, it.y);
        ++ahead;
      }
    }
  }
  wait();

  // Group mode (p.decode_group, a batch whose items would not fill the device's warps): item 8 g + w is the w-th
  // eighth of the pages of group g = (sequence, KV head); a block takes whole groups -- g = block, block + n_blocks,
  // ... -- its eight warps one slice each, and their partial results meet in the block's shared memory instead of in
  // global memory behind a counter.  Every warp of the block goes through the same barriers whatever happens to it.
  const bool group_mode = p.decode_group != 0;
  bool first_round = true;
  for (int round = 0;; ++round) {
    if (!first_round) {
      if (group_mode) {
        item = worker ? (block + round * n_blocks) * DC_WARPS + warp : p.n_decode_items;
      } else {
        if (lane == 0) item = n_blocks * DC_WARPS + atomicAdd(counters + 1, 1);
        item = __shfl_sync(0xffffffffu, item, 0);
      }
    }
    if (item >= p.n_decode_items || (!group_mode && *abort_flag)) break;
    // one 32-byte record: {decode row, kv head, first key, end key} {seq, token row, the group's first partial slot,
    // splits | index within the group << 16}: the queue hands the items out longest first, the partials of a group
    // stay in key order
    if (!first_round) {
      it = reinterpret_cast<const int4*>(p.decode_items)[2 * item];
      dr = reinterpret_cast<const int4*>(p.decode_items)[2 * item + 1];
      ahead = 0;
    }
    const int drow = it.x, hk = it.y, k0 = it.z, k1 = it.w;
    const int seq = dr.x, tok = dr.y, splits = dr.w & 0xffff, part = dr.z + (dr.w >> 16);
    const int n_pages = (k1 - k0 + 15) >> 4;
    // the item's page ids, one per lane, fetched with a single load: reading the block table page by page
    // would put one dependent round trip to memory in front of every request
    if (!first_round) {
      const int32_t* table = p.block_tables + size_t(seq) * p.max_pages_per_seq + (k0 >> 4);
      my_page = lane < n_pages ? table[lane] : 0;      // the planner keeps items within 32 pages
    }
    first_round = false;
#pragma unroll
    for (int pi = 0; pi < DC_STAGES - 1; ++pi) {
      const int page = __shfl_sync(0xffffffffu, my_page, pi);
      if (lane == 0 && pi >= ahead && pi < n_pages) issue(page, hk);
    }

    // Q fragments straight from global memory: rows = query heads hk*G .. hk*G + G - 1 of the new token
    const __nv_bfloat16* qrow = p.q + size_t(tok) * q_dim + size_t(hk) * G * DH;
    const int ra = lane >> 2, rb = ra + 8;
    uint32_t qf[DH / 16][4];
#pragma unroll
    for (int ks = 0; ks < DH / 16; ++ks) {
      const int c = ks * 16 + 2 * (lane & 3);
      // (read through the L2: in the one-launch small step another block of the same launch wrote q)
      qf[ks][0] = ra < G ? __ldcg(reinterpret_cast<const uint32_t*>(qrow + ra * DH + c)) : 0u;
      qf[ks][1] = rb < G ? __ldcg(reinterpret_cast<const uint32_t*>(qrow + rb * DH + c)) : 0u;
      qf[ks][2] = ra < G ? __ldcg(reinterpret_cast<const uint32_t*>(qrow + ra * DH + c + 8)) : 0u;
      qf[ks][3] = rb < G ? __ldcg(reinterpret_cast<const uint32_t*>(qrow + rb * DH + c + 8)) : 0u;
    }
    float o_acc[DH / 8][4];
#pragma unroll
    for (int j = 0; j < DH / 8; ++j) o_acc[j][0] = o_acc[j][1] = o_acc[j][2] = o_acc[j][3] = 0.f;
    float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
    bool ok = true;

    for (int pi = 0; pi < n_pages; ++pi) {
      // the slot read in the previous iteration is free: keep DC_STAGES - 1 pages in flight
      const int page_ahead = __shfl_sync(0xffffffffu, my_page, (pi + DC_STAGES - 1) & 31);
      if (lane == 0 && pi + DC_STAGES - 1 < n_pages) issue(page_ahead, hk);
      const uint32_t st = consumed % DC_STAGES;
      ok = mbar_wait(&full[st], (consumed / DC_STAGES) & 1, abort_flag, p.status);
      if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
      ++consumed;
      const uint32_t k_base = smem_u32(slots + st * SLOT_BYTES);
      const uint32_t v_base = k_base + G_::PAGE_BYTES;
      const int n_valid = k1 - (k0 + pi * 16);            // keys of this page that belong to the item
      float sc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
      for (int ks = 0; ks < DH / 16; ++ks) {
        uint32_t kf[4];
        const int kk = (lane & 7) + (lane >> 4) * 8, cc = 2 * ks + ((lane >> 3) & 1);
        ldmatrix_x4(kf, k_base + kv_off(kk, cc));
        mma_bf16_16816(sc[0], qf[ks], kf[0], kf[1]);
        mma_bf16_16816(sc[1], qf[ks], kf[2], kf[3]);
      }
      float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v = sc[j][e] * scale_log2;
          if (8 * j + 2 * (lane & 3) + (e & 1) >= n_valid) v = -INFINITY;
          sc[j][e] = v;
        }
        mx_a = fmaxf(mx_a, fmaxf(sc[j][0], sc[j][1]));
        mx_b = fmaxf(mx_b, fmaxf(sc[j][2], sc[j][3]));
      }
      mx_a = quad_max(mx_a);
      mx_b = quad_max(mx_b);
      const float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);
      const float al_a = exp2f(m_a - mn_a), al_b = exp2f(m_b - mn_b);
      // the running maxima settle after a few pages: skip the rescale of O when no row's maximum moved
      const bool rescale = __any_sync(0xffffffffu, mn_a != m_a || mn_b != m_b);
      m_a = mn_a;
      m_b = mn_b;
      float sum_a = 0.f, sum_b = 0.f;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        sc[j][0] = exp2f(sc[j][0] - mn_a);
        sc[j][1] = exp2f(sc[j][1] - mn_a);
        sc[j][2] = exp2f(sc[j][2] - mn_b);
        sc[j][3] = exp2f(sc[j][3] - mn_b);
        sum_a += sc[j][0] + sc[j][1];
        sum_b += sc[j][2] + sc[j][3];
      }
      l_a = l_a * al_a + sum_a;
      l_b = l_b * al_b + sum_b;
      if (rescale) {
#pragma unroll
        for (int j = 0; j < DH / 8; ++j) {
          o_acc[j][0] *= al_a; o_acc[j][1] *= al_a;
          o_acc[j][2] *= al_b; o_acc[j][3] *= al_b;
        }
      }
      uint32_t pf[4];
      pf[0] = pack_bf16(sc[0][0], sc[0][1]);
      pf[1] = pack_bf16(sc[0][2], sc[0][3]);
      pf[2] = pack_bf16(sc[1][0], sc[1][1]);
      pf[3] = pack_bf16(sc[1][2], sc[1][3]);
#pragma unroll
      for (int dp = 0; dp < DH / 16; ++dp) {
        uint32_t vf[4];
        const int kk = (lane & 7) + ((lane >> 3) & 1) * 8, cc = 2 * dp + (lane >> 4);
        ldmatrix_x4_trans(vf, v_base + kv_off(kk, cc));
        if (n_valid < 16) {
          const int k = 2 * (lane & 3);
          vf[0] = mask_v(vf[0], k, n_valid);
          vf[1] = mask_v(vf[1], k + 8, n_valid);
          vf[2] = mask_v(vf[2], k, n_valid);
          vf[3] = mask_v(vf[3], k + 8, n_valid);
        }
        mma_bf16_16816(o_acc[2 * dp], pf, vf[0], vf[1]);
        mma_bf16_16816(o_acc[2 * dp + 1], pf, vf[2], vf[3]);
      }
      __syncwarp();                         // every lane is done with this slot before lane 0 refills it
    }
    if (!ok && !group_mode) break;

    l_a = quad_sum(l_a);
    l_b = quad_sum(l_b);
    __nv_bfloat16* orow = p.o + size_t(tok) * q_dim + size_t(hk) * G * DH;
    if (group_mode) {
      // this slice's partial into the warp's own (now idle) page ring: [16 rows][DH] unnormalised output, then
      // [16 rows] (max, sum)
      float* po = reinterpret_cast<float*>(slots);
      float2* pml = reinterpret_cast<float2*>(slots + 16 * DH * 4);
#pragma unroll
      for (int j = 0; j < DH / 8; ++j) {
        const int col = 8 * j + 2 * (lane & 3);
        if (ra < G) *reinterpret_cast<float2*>(po + ra * DH + col) = make_float2(o_acc[j][0], o_acc[j][1]);
        if (rb < G) *reinterpret_cast<float2*>(po + rb * DH + col) = make_float2(o_acc[j][2], o_acc[j][3]);
      }
      if ((lane & 3) == 0) {
        if (ra < G) pml[ra] = make_float2(m_a, l_a);
        if (rb < G) pml[rb] = make_float2(m_b, l_b);
      }
      const bool failed = __syncthreads_or(!ok) != 0;      // the same answer in every warp of the block
      if (!failed) {
        // the eight partials are merged in slice order by the whole block: a thread per pair of output columns
        const bool f16 = p.o_f16 != 0;
        for (int e = threadIdx.x; e < G * (DH / 2); e += blockDim.x) {
          const int g = e / (DH / 2), col = 2 * (e - g * (DH / 2));
          float mm = -INFINITY;
#pragma unroll
          for (int w = 0; w < DC_WARPS; ++w)
            mm = fmaxf(mm, reinterpret_cast<const float2*>(smem + w * DC_STAGES * SLOT_BYTES + 16 * DH * 4)[g].x);
          float ll = 0.f, o0 = 0.f, o1 = 0.f;
#pragma unroll
          for (int w = 0; w < DC_WARPS; ++w) {
            const uint8_t* base = smem + w * DC_STAGES * SLOT_BYTES;
            const float2 ml = reinterpret_cast<const float2*>(base + 16 * DH * 4)[g];
            const float f = exp2f(ml.x - mm);                 // 0 for an empty slice (max = -inf)
            const float2 v = *reinterpret_cast<const float2*>(reinterpret_cast<const float*>(base) + g * DH + col);
            ll += f * ml.y;
            o0 += f * v.x;
            o1 += f * v.y;
          }
          const float inv = 1.f / ll;
          if (f16) {
            const float v2[2] = {o0, o1};
            note_f16_saturation(v2, p.status, inv);
          }
          *reinterpret_cast<uint32_t*>(orow + g * DH + col) = pack_act(o0 * inv, o1 * inv, f16);
        }
      }
      // the rings go back to the copy engine: order these generic-proxy accesses before its next writes
      fence_proxy_async();
      __syncthreads();
      if (failed) break;
      continue;
    }
    if (splits == 1) {
      // the whole key range was this item: normalise and write the output rows directly
      const float inv_a = 1.f / l_a, inv_b = 1.f / l_b;
      if (p.o_f16) {                        // saturation report of the fp16 output (see note_f16_saturation)
        float mx_oa = 0.f, mx_ob = 0.f;
#pragma unroll
        for (int j = 0; j < DH / 8; ++j) {
          mx_oa = fmaxf(mx_oa, fmaxf(fabsf(o_acc[j][0]), fabsf(o_acc[j][1])));
          mx_ob = fmaxf(mx_ob, fmaxf(fabsf(o_acc[j][2]), fabsf(o_acc[j][3])));
        }
        if ((ra < G && mx_oa * inv_a > 65504.f) || (rb < G && mx_ob * inv_b > 65504.f)) {
          int c = 0;
#pragma unroll
          for (int j = 0; j < DH / 8; ++j) {
            if (ra < G) c += (fabsf(o_acc[j][0] * inv_a) > 65504.f) + (fabsf(o_acc[j][1] * inv_a) > 65504.f);
            if (rb < G) c += (fabsf(o_acc[j][2] * inv_b) > 65504.f) + (fabsf(o_acc[j][3] * inv_b) > 65504.f);
          }
          atomicAdd(p.status + 1, c);
        }
      }
#pragma unroll
      for (int j = 0; j < DH / 8; ++j) {
        const int col = 8 * j + 2 * (lane & 3);
        if (ra < G) *reinterpret_cast<uint32_t*>(orow + ra * DH + col) = pack_act(o_acc[j][0] * inv_a, o_acc[j][1] * inv_a, p.o_f16 != 0);
        if (rb < G) *reinterpret_cast<uint32_t*>(orow + rb * DH + col) = pack_act(o_acc[j][2] * inv_b, o_acc[j][3] * inv_b, p.o_f16 != 0);
      }
      continue;
    }
    // the item's partial: unnormalised output, running max (log2 domain) and sum, rows = query heads
    float* po = p.part_o + size_t(part) * 16 * DH;
    float* pml = p.part_ml + size_t(part) * 16 * 2;
#pragma unroll
    for (int j = 0; j < DH / 8; ++j) {
      const int col = 8 * j + 2 * (lane & 3);
      if (ra < G) *reinterpret_cast<float2*>(po + ra * DH + col) = make_float2(o_acc[j][0], o_acc[j][1]);
      if (rb < G) *reinterpret_cast<float2*>(po + rb * DH + col) = make_float2(o_acc[j][2], o_acc[j][3]);
    }
    if ((lane & 3) == 0) {
      if (ra < G) { pml[ra * 2] = m_a; pml[ra * 2 + 1] = l_a; }
      if (rb < G) { pml[rb * 2] = m_b; pml[rb * 2 + 1] = l_b; }
    }
    // The warp that completes the last split of a (sequence, KV head) merges all of its splits, always in
    // split order, so the result does not depend on which warp that is.
    __threadfence();
    __syncwarp();
    int* done = p.group_done + drow * p.n_kv_heads + hk;
    int last = 0;
    if (lane == 0) last = atomicAdd(done, 1) == splits - 1;
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) {
      __threadfence();
      const int first = dr.z;
      if (G <= 8) merge_group<DH, 4, DC_STAGES * SLOT_BYTES>(p.part_o, p.part_ml, slots, first, splits, G, lane, orow, p.o_f16 != 0, p.status);
      else merge_group<DH, 2, DC_STAGES * SLOT_BYTES>(p.part_o, p.part_ml, slots, first, splits, G, lane, orow, p.o_f16 != 0, p.status);
      if (lane == 0) *done = 0;             // ready for the next launch
    }
  }
  __syncthreads();
  if (*abort_flag) drain_after_abort();
}


}  // namespace
}  // namespace hs
