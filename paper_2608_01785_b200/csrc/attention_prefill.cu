// Causal GQA attention for prefill chunks on the 5th-generation tensor cores.
//
//   work item   (sequence, KV head, tile of Mt tokens), Mt = 128 / G rounded down to a multiple of 8.  The G
//               query heads that share the KV head are stacked head-major as rows of one 128-row tile
//               (row = head * Mt + token), so K and V are streamed once per KV head.
//   per block   of 64 keys:  S = Q K^T (tcgen05.mma, M128 N64, fp32 in tensor memory)  ->  softmax warps
//               (one thread per row: no shuffles) read S, scale, mask by selection, keep the running max and
//               sum in the log2 domain, write P as bf16 into a swizzled shared-memory tile  ->  O_blk = P V
//               (tcgen05.mma, M128 N=Dh, V used in place as an MN-major operand)  ->  the same threads fold
//               O_blk into fp32 registers: o = o * exp2(m_old - m_new) + O_blk.
//   pipeline    S, P and O_blk are double buffered, so the MMA warp computes S of block j+1 while the
//               softmax warps work on block j; K/V pages arrive by TMA in a 4-stage ring ([half][page][16][64]
//               tiles with the 128-byte swizzle, the K tile being a K-major and the V tile an MN-major
//               operand); the producer owns the work queue and runs ahead across items.
//   roles       warps 0..3 softmax / correction (thread = row = TMEM lane), warp 4 TMA producer, warp 5 MMA
//               issuer and TMEM owner.
// Keys past the end of a sequence are masked by selection on the key index, and the matching V rows are
// zeroed in shared memory before the P V product, so arbitrary bytes in unused cache slots cannot reach
// the output.  An item's result does not depend on which block ran it: outputs are budget independent.
#include <math.h>

#include "kernels.h"
#include "ptx.cuh"

namespace hs {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int PF_THREADS = 192, PF_STAGES = 3, PF_KEYS = 64;
constexpr int TMEM_COLS = 512;

template <int DH>
struct Geom {
  static constexpr int HALVES = DH / 64;
  static constexpr int Q_BYTES = HALVES * 16384;        // [half][128 rows][128 B]
  static constexpr int KV_BYTES = HALVES * 8192;        // K (or V) of one stage: [half][4 pages][16 keys][128 B]
  static constexpr int STAGE_BYTES = 2 * KV_BYTES;
  static constexpr int P_BYTES = 16384;                 // [128 rows][64 keys] bf16
  static constexpr int SMEM = 1024 + 2 * Q_BYTES + PF_STAGES * STAGE_BYTES + 2 * P_BYTES + 512;
  // tensor-memory columns
  static constexpr int S0 = 0, O0 = 128;                // S buffers at 0 / 64, O_blk buffers at 128 / 128 + DH
};

struct Barriers {
  uint64_t q_full[2], q_empty[2];
  uint64_t kv_full[PF_STAGES], kv_empty[PF_STAGES];
  uint64_t s_full[2], s_empty[2], p_full[2], o_full[2], o_empty[2];
  uint64_t ring_full[2], ring_empty[2];
  int ring_item[2];
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ int pool_row(const AttnParams& p, int kv, int page, int hk) {
  return (((p.layer * 2 + kv) * p.num_pages + page) * p.n_kv_heads + hk) * 16;
}
// 2^x on the special-function unit (ex2.approx: exact 0 for -inf, relative error about 2^-22).
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// MN-major bf16 operand with the 128-byte swizzle: atoms of 64 (MN, contiguous) x 8 (K) elements;
// lbo = bytes between atoms along MN, sbo = bytes between atoms along K.
__device__ __forceinline__ uint64_t umma_desc_mnmajor_sw128(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((smem_addr & 0x3ffffu) >> 4);
  d |= static_cast<uint64_t>(lbo >> 4) << 16;
  d |= static_cast<uint64_t>(sbo >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

template <int DH>
__global__ void __launch_bounds__(PF_THREADS, 1) attn_prefill_kernel(const __grid_constant__ AttnParams p) {
  using G_ = Geom<DH>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_smem = smem;
  uint8_t* stages = q_smem + 2 * G_::Q_BYTES;       // two Q tiles: the next item's tile loads early
  uint8_t* p_smem = stages + PF_STAGES * G_::STAGE_BYTES;
  Barriers* bar = reinterpret_cast<Barriers*>(p_smem + 2 * G_::P_BYTES);
  volatile int* abort_flag = &bar->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  log_smid(p.smid_log);
  const int G = p.n_q_heads / p.n_kv_heads;
  const int Mt = p.prefill_tokens;
  const int q_dim = p.n_q_heads * DH;
  const float scale_log2 = kLog2e / sqrtf(float(DH));

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bar->q_full[i], 1);
      mbar_init(&bar->q_empty[i], 1);
    }
    for (int i = 0; i < PF_STAGES; ++i) {
      mbar_init(&bar->kv_full[i], 1);
      mbar_init(&bar->kv_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bar->s_full[i], 1);
      mbar_init(&bar->s_empty[i], 128);
      mbar_init(&bar->p_full[i], 128);
      mbar_init(&bar->o_full[i], 1);
      mbar_init(&bar->o_empty[i], 128);
      mbar_init(&bar->ring_full[i], 1);
      mbar_init(&bar->ring_empty[i], 5);    // four softmax warps + the MMA warp
    }
    bar->abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&p.tm_kv);
    tma_prefetch_desc(&p.tm_q);
  }
  if (warp == 5) {
    tmem_alloc(&bar->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = bar->tmem_base;
  griddep_wait();
  griddep_launch_dependents();

  int rs = 0;
  uint32_t rph = 0;       // item ring slot / phase
  uint32_t gblk = 0;      // key blocks processed so far by this thread's role, over all items
  uint32_t n_items_seen = 0;

  if (warp == 4) {
    // =========================================================== TMA producer ==
    if (lane == 0) {
      for (;;) {
        if (!mbar_wait(&bar->ring_empty[rs], rph ^ 1, abort_flag, p.status)) break;
        const int item = atomicAdd(p.counters, 1);
        bar->ring_item[rs] = item;
        mbar_arrive(&bar->ring_full[rs]);
        if (++rs == 2) { rs = 0; rph ^= 1; }
        if (item >= p.n_prefill_items) break;
        const int4 it = reinterpret_cast<const int4*>(p.prefill_items)[item];
        const int seq = it.x, hk = it.y, tok_begin = it.z, n_tok = it.w;
        const int tok0 = p.seq_tok0[seq] + tok_begin;
        const int n_keys = p.seq_ctx[seq] + (p.bidirectional ? p.seq_qlen[seq] : tok_begin + n_tok);
        const int n_kblocks = (n_keys + PF_KEYS - 1) / PF_KEYS;
        const int32_t* table = p.block_tables + size_t(seq) * p.max_pages_per_seq;
        // Q tile: one box of Mt token rows x 64 columns per (head, half)
        const uint32_t qb = n_items_seen & 1;
        if (!mbar_wait(&bar->q_empty[qb], ((n_items_seen >> 1) & 1) ^ 1, abort_flag, p.status)) break;
        mbar_expect_tx(&bar->q_full[qb], G * G_::HALVES * Mt * 128);
        for (int g = 0; g < G; ++g)
          for (int h = 0; h < G_::HALVES; ++h)
            tma_load_2d(q_smem + qb * G_::Q_BYTES + h * 16384 + g * Mt * 128, &p.tm_q, &bar->q_full[qb],
                        (hk * G + g) * DH + h * 64, tok0);
        ++n_items_seen;
        bool ok = true;
        for (int kb = 0; kb < n_kblocks; ++kb, ++gblk) {
          const int s = gblk % PF_STAGES;
          if (!mbar_wait(&bar->kv_empty[s], ((gblk / PF_STAGES) & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
          const int rem = n_keys - kb * PF_KEYS;
          const int np = rem >= PF_KEYS ? 4 : (rem + 15) >> 4;
          uint8_t* st = stages + s * G_::STAGE_BYTES;
          mbar_expect_tx(&bar->kv_full[s], np * 2 * G_::HALVES * 2048);
          for (int w = 0; w < np; ++w) {
            const int page = table[kb * 4 + w];
            const int krow = pool_row(p, 0, page, hk), vrow = pool_row(p, 1, page, hk);
            for (int h = 0; h < G_::HALVES; ++h) {
              tma_load_2d(st + h * 8192 + w * 2048, &p.tm_kv, &bar->kv_full[s], h * 64, krow);
              tma_load_2d(st + G_::KV_BYTES + h * 8192 + w * 2048, &p.tm_kv, &bar->kv_full[s], h * 64, vrow);
            }
          }
        }
        if (!ok) break;
      }
    }
  } else if (warp == 5) {
    // ============================================================= MMA issuer ==
    if (lane == 0) {
      constexpr uint32_t idesc_s = umma_idesc_bf16_f32(128, PF_KEYS);
      constexpr uint32_t idesc_pv = umma_idesc_bf16_f32(128, DH) | (1u << 16);   // B (= V) is MN-major
      const uint32_t q_addr = smem_u32(q_smem), st_addr = smem_u32(stages), p_addr = smem_u32(p_smem);
      // O_blk(buffer of block b) = P(buffer) * V(stage of block b)
      auto issue_pv = [&](uint32_t b) -> bool {
        const uint32_t buf = b & 1, bph = (b >> 1) & 1, s = b % PF_STAGES;
        if (!mbar_wait(&bar->p_full[buf], bph, abort_flag, p.status)) return false;
        if (!mbar_wait(&bar->o_empty[buf], bph ^ 1, abort_flag, p.status)) return false;
        tc_fence_after_sync();
        const uint32_t v_addr = st_addr + s * G_::STAGE_BYTES + G_::KV_BYTES;
#pragma unroll
        for (int pg = 0; pg < 4; ++pg) {      // 16 keys (one page) per MMA
          const uint64_t a = umma_desc_kmajor_sw128(p_addr + buf * G_::P_BYTES) + 2 * pg;
          const uint64_t bdesc = umma_desc_mnmajor_sw128(v_addr + pg * 2048, 8192, 1024);
          umma_bf16(tmem + G_::O0 + buf * DH, a, bdesc, idesc_pv, pg != 0);
        }
        umma_commit(&bar->o_full[buf]);
        umma_commit(&bar->kv_empty[s]);
        return true;
      };
      for (;;) {
        if (!mbar_wait(&bar->ring_full[rs], rph, abort_flag, p.status)) break;
        const int item = bar->ring_item[rs];
        mbar_arrive(&bar->ring_empty[rs]);
        if (++rs == 2) { rs = 0; rph ^= 1; }
        if (item >= p.n_prefill_items) break;
        const int4 it = reinterpret_cast<const int4*>(p.prefill_items)[item];
        const int n_keys = p.seq_ctx[it.x] + (p.bidirectional ? p.seq_qlen[it.x] : it.z + it.w);
        const int n_kblocks = (n_keys + PF_KEYS - 1) / PF_KEYS;
        const uint32_t qb = n_items_seen & 1;
        if (!mbar_wait(&bar->q_full[qb], (n_items_seen >> 1) & 1, abort_flag, p.status)) break;
        ++n_items_seen;
        bool ok = true;
        for (int j = 0; j < n_kblocks && ok; ++j, ++gblk) {
          const uint32_t buf = gblk & 1, bph = (gblk >> 1) & 1, s = gblk % PF_STAGES;
          if (!mbar_wait(&bar->kv_full[s], (gblk / PF_STAGES) & 1, abort_flag, p.status)) { ok = false; break; }
          if (!mbar_wait(&bar->s_empty[buf], bph ^ 1, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after_sync();
          const uint32_t k_addr = st_addr + s * G_::STAGE_BYTES;
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks) {
            const uint64_t a = umma_desc_kmajor_sw128(q_addr + qb * G_::Q_BYTES + (ks >> 2) * 16384) + 2 * (ks & 3);
            const uint64_t b = umma_desc_kmajor_sw128(k_addr + (ks >> 2) * 8192) + 2 * (ks & 3);
            umma_bf16(tmem + G_::S0 + buf * PF_KEYS, a, b, idesc_s, ks != 0);
          }
          umma_commit(&bar->s_full[buf]);
          if (j == n_kblocks - 1) umma_commit(&bar->q_empty[qb]);   // this Q tile may be replaced once these are done
          if (j > 0) ok = issue_pv(gblk - 1);                      // overlaps the softmax of block j
        }
        if (!ok || !issue_pv(gblk - 1)) break;
      }
    }
  } else {
    // ================================================= softmax and correction ==
    const int r = threadIdx.x;                    // row of the tile = TMEM lane
    const uint32_t lane_base = uint32_t(warp * 32) << 16;
    for (;;) {
      bool ok = mbar_wait(&bar->ring_full[rs], rph, abort_flag, p.status);
      if (!__all_sync(0xffffffffu, ok)) break;
      const int item = bar->ring_item[rs];
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar->ring_empty[rs]);
      if (++rs == 2) { rs = 0; rph ^= 1; }
      if (item >= p.n_prefill_items) break;
      const int4 it = reinterpret_cast<const int4*>(p.prefill_items)[item];
      const int seq = it.x, hk = it.y, tok_begin = it.z, n_tok = it.w;
      const int tok0 = p.seq_tok0[seq] + tok_begin;
      const int pos0 = p.seq_ctx[seq] + tok_begin;
      const int n_keys = p.bidirectional ? p.seq_ctx[seq] + p.seq_qlen[seq] : pos0 + n_tok;
      const int n_kblocks = (n_keys + PF_KEYS - 1) / PF_KEYS;
      const int g = r / Mt, tok = r - g * Mt;
      const bool row_valid = g < G && tok < n_tok;
      // last key a row sees: its own position (padding rows behave like the last token), or the sequence's last key
      const int pos = p.bidirectional ? n_keys - 1 : pos0 + min(tok, n_tok - 1);

      float o_reg[DH];
#pragma unroll
      for (int e = 0; e < DH; ++e) o_reg[e] = 0.f;
      float m_run = -INFINITY, l_run = 0.f, alpha_prev = 0.f;
      uint32_t sreg[32], sreg2[32];

      // o = o * alpha + O_blk of block b
      auto correct = [&](uint32_t b, float alpha) -> bool {
        const uint32_t buf = b & 1, bph = (b >> 1) & 1;
        const bool w = mbar_wait(&bar->o_full[buf], bph, abort_flag, p.status);
        if (!__all_sync(0xffffffffu, w)) return false;
        tc_fence_after_sync();
#pragma unroll
        for (int c = 0; c < DH / 64; ++c) {
          tmem_ld32(tmem + lane_base + G_::O0 + buf * DH + c * 64, sreg);
          tmem_ld32(tmem + lane_base + G_::O0 + buf * DH + c * 64 + 32, sreg2);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            o_reg[c * 64 + e] = fmaf(o_reg[c * 64 + e], alpha, __uint_as_float(sreg[e]));
            o_reg[c * 64 + 32 + e] = fmaf(o_reg[c * 64 + 32 + e], alpha, __uint_as_float(sreg2[e]));
          }
        }
        tc_fence_before_sync();
        mbar_arrive(&bar->o_empty[buf]);
        return true;
      };

      for (int j = 0; j < n_kblocks; ++j, ++gblk) {
        const uint32_t buf = gblk & 1, bph = (gblk >> 1) & 1;
        ok = mbar_wait(&bar->s_full[buf], bph, abort_flag, p.status);
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
        tc_fence_after_sync();
        const int key0 = j * PF_KEYS;
        // both halves of the row in flight, one wait
        tmem_ld32(tmem + lane_base + G_::S0 + buf * PF_KEYS, sreg);
        tmem_ld32(tmem + lane_base + G_::S0 + buf * PF_KEYS + 32, sreg2);
        tmem_ld_wait();
        tc_fence_before_sync();
        mbar_arrive(&bar->s_empty[buf]);
        if (key0 + PF_KEYS - 1 > pos) {               // this row does not see every key of the block
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            if (key0 + e > pos) sreg[e] = 0xff800000u;          // -inf
            if (key0 + 32 + e > pos) sreg2[e] = 0xff800000u;
          }
        }
        float mx = -INFINITY;
#pragma unroll
        for (int e = 0; e < 32; ++e) mx = fmaxf(mx, fmaxf(__uint_as_float(sreg[e]), __uint_as_float(sreg2[e])));
        // running max kept on the raw scores; the 1/sqrt(Dh) * log2(e) scale is folded into the exponent
        const float m_new = fmaxf(m_run, mx);
        const float alpha = fast_exp2((m_run - m_new) * scale_log2);
        const float neg_ms = -m_new * scale_log2;
        m_run = m_new;
        float sum = 0.f;
        uint8_t* prow = p_smem + buf * G_::P_BYTES + r * 128;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          float e8[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const uint32_t raw = u < 4 ? sreg[u * 8 + e] : sreg2[(u - 4) * 8 + e];
            e8[e] = fast_exp2(fmaf(__uint_as_float(raw), scale_log2, neg_ms));
            sum += e8[e];
          }
          uint4 w;
          w.x = pack_bf16(e8[0], e8[1]);
          w.y = pack_bf16(e8[2], e8[3]);
          w.z = pack_bf16(e8[4], e8[5]);
          w.w = pack_bf16(e8[6], e8[7]);
          *reinterpret_cast<uint4*>(prow + ((u ^ (r & 7)) << 4)) = w;
        }
        l_run = l_run * alpha + sum;
        // ragged last block: V rows of keys that do not exist must not carry stray NaN / Inf bits
        const int n_valid = n_keys - key0;
        if (n_valid < PF_KEYS) {
          const uint32_t s = gblk % PF_STAGES;
          const bool w = mbar_wait(&bar->kv_full[s], (gblk / PF_STAGES) & 1, abort_flag, p.status);
          if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
          uint8_t* vst = stages + s * G_::STAGE_BYTES + G_::KV_BYTES;
          const int n_units = (PF_KEYS - n_valid) * G_::HALVES * 8;
          for (int idx = r; idx < n_units; idx += 128) {
            const int u = idx & 7, h = (idx >> 3) % G_::HALVES, k = n_valid + (idx >> 3) / G_::HALVES;
            *reinterpret_cast<uint4*>(vst + h * 8192 + (k >> 4) * 2048 + (k & 15) * 128 + (u << 4)) =
                make_uint4(0, 0, 0, 0);
          }
        }
        fence_proxy_async();
        mbar_arrive(&bar->p_full[buf]);
        if (j > 0 && !correct(gblk - 1, alpha_prev)) { ok = false; break; }
        alpha_prev = alpha;
      }
      if (!ok) break;
      if (!correct(gblk - 1, alpha_prev)) break;
      if (row_valid) {
        const float inv = 1.f / l_run;
        const bool f16 = p.o_f16 != 0;
        __nv_bfloat16* dst = p.o + size_t(tok0 + tok) * q_dim + (hk * G + g) * DH;
#pragma unroll
        for (int u = 0; u < DH / 8; ++u) {
          uint4 w;
          w.x = pack_act(o_reg[u * 8 + 0] * inv, o_reg[u * 8 + 1] * inv, f16);
          w.y = pack_act(o_reg[u * 8 + 2] * inv, o_reg[u * 8 + 3] * inv, f16);
          w.z = pack_act(o_reg[u * 8 + 4] * inv, o_reg[u * 8 + 5] * inv, f16);
          w.w = pack_act(o_reg[u * 8 + 6] * inv, o_reg[u * 8 + 7] * inv, f16);
          *reinterpret_cast<uint4*>(dst + u * 8) = w;
        }
      }
    }
  }

  // --------------------------------------------------------------- teardown --
  __syncwarp();
  if (*abort_flag) drain_after_abort();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

template <int DH>
constexpr int pf_smem_bytes() {
  return Geom<DH>::SMEM > kMinSmemBytes ? Geom<DH>::SMEM : kMinSmemBytes;
}

}  // namespace

cudaError_t attention_prefill_set_attributes() {
  cudaError_t e = set_kernel_smem(attn_prefill_kernel<64>, pf_smem_bytes<64>());
  if (e != cudaSuccess) return e;
  return set_kernel_smem(attn_prefill_kernel<128>, pf_smem_bytes<128>());
}

cudaError_t launch_attention_prefill(const AttnParams& p, int sm_budget, cudaStream_t stream) {
  if (p.n_prefill_items <= 0) return cudaSuccess;
  const int grid = p.n_prefill_items < sm_budget ? p.n_prefill_items : sm_budget;
  if (p.head_dim == 128)
    return launch_step_kernel(attn_prefill_kernel<128>, grid, PF_THREADS, pf_smem_bytes<128>(), stream, p.overlap != 0, p);
  else
    return launch_step_kernel(attn_prefill_kernel<64>, grid, PF_THREADS, pf_smem_bytes<64>(), stream, p.overlap != 0, p);
}

}  // namespace hs
