// Causal GQA attention for prefill chunks on the 5th-generation tensor cores.
//
//   work item   (sequence, KV head, up to 2 Mt consecutive tokens), Mt = 128 / G rounded down to a multiple of 8.
//               The item is two Q tiles: tile A holds its first Mt tokens, tile B the rest.  In a tile the G query
//               heads that share the KV head are stacked head-major as rows of a 128-row tile (row = head * Mt +
//               token).  Both tiles read the same K / V blocks, which are staged once for the two of them.
//   per block   of 64 keys and per tile:  S = Q K^T (tcgen05.mma, M128 N64, fp32 in tensor memory)  ->  the tile's
//               softmax warp group (one thread per row: no shuffles) reads S, masks by selection, exponentiates
//               in the log2 domain against a per-row reference maximum, writes P as bf16 back into tensor memory,
//               over the first half of the S buffer it has just read (tcgen05.st: row = lane, two keys per
//               32-bit column)  ->  O += P V (tcgen05.mma with the A operand in tensor memory, M128 N = Dh, V used
//               in place as an MN-major operand from shared memory).  An MMA whose operands both come from shared
//               memory is bound by the operand fetch (about 64 bytes per clock and SM); taking P from tensor
//               memory halves the bytes of the P V product.  O stays in tensor memory for the whole item; it is
//               read once, at the item's end.
//   reference   A row's reference maximum follows its running maximum lazily: it moves only when the running
//   maximum     maximum exceeds it by more than 8 (in log2 units, a factor of 256), and only then is the row of O
//               rescaled (tcgen05.ld / multiply / tcgen05.st by the softmax threads, while no P V product of the
//               tile is in flight).  P and the running sum use the same reference, so the quotient O / l at the
//               end is exact whatever reference was used; values stay far inside the range of bf16 and fp32.
//   pipeline    two tiles x two S buffers: while one tile's warp group exponentiates, the tensor core works on the
//               other tile's products.  The tensor core runs its instructions in issue order, which is what makes
//               the overlay safe: S of block j + 2 is issued after the P V product of block j, whose P it replaces.  K and V blocks arrive by TMA in two rings of their own
//               ([half][page][16][64] tiles with the 128-byte swizzle, the K tile being a K-major and the V tile an
//               MN-major operand): a K slot is free again as soon as the block's scores are computed, a V slot
//               after its P V products.  The producers own the work queue and run ahead across items.
//   roles       warps 0..3 softmax of tile A, warps 4..7 softmax of tile B (thread = row = TMEM lane), warp 8 and
//               warps 11..13 TMA producers, warp 9 MMA issuer of tile A and TMEM owner, warp 10 MMA issuer of tile B.
// Keys past the end of a sequence are masked by selection on the key index, and the matching V rows are
// zeroed in shared memory before the P V product, so arbitrary bytes in unused cache slots cannot reach
// the output.  An item's result does not depend on which block ran it: outputs are budget independent.
#include <math.h>

#include "kernels.h"
#include "ptx.cuh"

namespace hs {
namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int PF_THREADS = 448, PF_KEYS = 64;
constexpr int PF_KSTAGES = 4, PF_VSTAGES = 4;
constexpr int TMEM_COLS = 512;
constexpr float kRefSlack = 8.f;   // log2 units by which a row's running maximum may exceed its reference

template <int DH>
struct Geom {
  static constexpr int HALVES = DH / 64;
  static constexpr int Q_BYTES = HALVES * 16384;        // one tile: [half][128 rows][128 B]
  static constexpr int KV_BYTES = HALVES * 8192;        // K (or V) of one block: [half][4 pages][16 keys][128 B]
  static constexpr int SMEM = 1024 + 2 * Q_BYTES + (PF_KSTAGES + PF_VSTAGES) * KV_BYTES + 1024;
  // tensor-memory columns: S(tile, buffer) at tile * 128 + buffer * 64, P(tile, buffer) over its first 32 columns;
  // O(tile) at 256 + tile * DH
  static constexpr int S0 = 0, O0 = 256;
};
static_assert(Geom<128>::SMEM <= 227 * 1024, "fits one SM");

// Geometry of one item, the same in every role.
struct ItemView {
  int seq, hk, tok_begin, n_tok;     // the item record
  int tok0, pos0, ctx;               // first token row of tile A, its absolute position, cached tokens
  int n_tok_t[2];                    // tokens of tile A / B (0 = tile absent)
  int n_keys;                        // keys the item's K / V blocks cover (valid cache rows)
  int nblk_t[2], nblk;               // key blocks per tile and of the item
};
struct Barriers {
  uint64_t q_full, q_empty;
  uint64_t k_full[PF_KSTAGES], k_empty[PF_KSTAGES], v_full[PF_VSTAGES], v_empty[PF_VSTAGES];
  uint64_t s_full[2][2], p_full[2][2], o_full[2][2];
  uint64_t ring_full[2], ring_empty[2];
  int ring_item[2];
  ItemView ring_view[2];          // the item's geometry, worked out once by the producer
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(Barriers) <= 1024, "barrier block");

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
// D[tmem] (+)= A[tmem] * B[smem]^T: the A operand (M rows = lanes, 16 K elements = 8 columns of packed pairs) is read
// from tensor memory; one thread issues for the block.
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}\n"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// An item's geometry from its 32-byte record {seq, kv head, first token, tokens} {cached tokens of the sequence, token
// row of the sequence's first new token, new tokens of the sequence, -}.
__device__ __forceinline__ ItemView view_item(const AttnParams& p, const int4& it, const int4& sq, int Mt) {
  ItemView v;
  v.seq = it.x; v.hk = it.y; v.tok_begin = it.z; v.n_tok = it.w;
  v.ctx = sq.x;
  v.tok0 = sq.y + v.tok_begin;
  v.pos0 = v.ctx + v.tok_begin;
  v.n_tok_t[0] = min(v.n_tok, Mt);
  v.n_tok_t[1] = v.n_tok - v.n_tok_t[0];
  const int all = v.ctx + sq.z;
  v.n_keys = p.bidirectional ? all : v.pos0 + v.n_tok;
  const int keys_a = p.bidirectional ? all : v.pos0 + v.n_tok_t[0];
  v.nblk_t[0] = (keys_a + PF_KEYS - 1) / PF_KEYS;
  v.nblk_t[1] = v.n_tok_t[1] > 0 ? (v.n_keys + PF_KEYS - 1) / PF_KEYS : 0;
  v.nblk = max(v.nblk_t[0], v.nblk_t[1]);
  return v;
}

template <int DH>
__global__ void __launch_bounds__(PF_THREADS, 1) attn_prefill_kernel(const __grid_constant__ AttnParams p) {
  using G_ = Geom<DH>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* q_smem = smem;                                   // tile A then tile B
  uint8_t* k_smem = q_smem + 2 * G_::Q_BYTES;
  uint8_t* v_smem = k_smem + PF_KSTAGES * G_::KV_BYTES;
  Barriers* bar = reinterpret_cast<Barriers*>(v_smem + PF_VSTAGES * G_::KV_BYTES);
  volatile int* abort_flag = &bar->abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  log_smid(p.smid_log);
  const int G = p.n_q_heads / p.n_kv_heads;
  const int Mt = p.prefill_tokens;
  const int q_dim = p.n_q_heads * DH;
  const float scale_log2 = kLog2e / sqrtf(float(DH));

  if (threadIdx.x == 0) {
    mbar_init(&bar->q_full, 1);
    mbar_init(&bar->q_empty, 2);              // one arrival per MMA thread
    for (int i = 0; i < PF_KSTAGES; ++i) { mbar_init(&bar->k_full[i], 2); mbar_init(&bar->k_empty[i], 2); }
    for (int i = 0; i < PF_VSTAGES; ++i) { mbar_init(&bar->v_full[i], 2); mbar_init(&bar->v_empty[i], 2); }
    for (int t = 0; t < 2; ++t) {
      for (int i = 0; i < 2; ++i) {
        mbar_init(&bar->s_full[t][i], 1);
        mbar_init(&bar->p_full[t][i], 128);
        mbar_init(&bar->o_full[t][i], 1);
      }
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bar->ring_full[i], 1);
      mbar_init(&bar->ring_empty[i], 13);     // eight softmax warps, two MMA warps, three further producers
    }
    bar->abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&p.tm_kv);
    tma_prefetch_desc(&p.tm_q);
  }
  if (warp == 9) {
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
  uint32_t n_items_seen = 0;
  uint32_t blk_base = 0;  // key blocks of all earlier items of this thread block (K / V ring position)

  if (warp == 8 || warp >= 11) {
    // ========================================================== TMA producers ==
    // Four warps share the page requests (a bulk tensor copy costs its issuing thread well over a hundred cycles,
    // and a 64-key block needs sixteen of them: one thread could not keep up with the tensor core): producer 0
    // (warp 8) owns the work queue, loads the Q tiles and pages 0, 1 of every K block; producer 1 pages 2, 3 of K;
    // producers 2 and 3 the same halves of V.  Lane 0 of each waits and issues; the whole warp fetches page ids:
    // lane l holds the id of page 32 c + l of the item for the current chunk c of 8 key blocks (one coalesced load per
    // chunk, requested a chunk ahead), so that no round trip to the block table stands in front of a page request.
    const int pi = warp == 8 ? 0 : warp - 10;           // producer index 0..3
    const int kv = pi >> 1, w0 = (pi & 1) * 2;          // K or V; first of its two pages in a block
    // The lead producer's lane 0 asks the work queue for the next item while it still has a few key blocks of the
    // current one to request, and for that item's record two blocks later -- so that neither the atomic nor the
    // record's round trip stands between two items (with items of one key block those two and the sequence's fields,
    // now part of the record, were most of an item's time).  Asking earlier -- at the item's start -- would hand the
    // items out before anybody knows which blocks finish early.  A block's first item is its index in the grid.
    int q_next = int(blockIdx.x);                                   // lane 0 of the lead: the next item's queue index
    int4 rec_a = make_int4(0, 0, 0, 0), rec_b = rec_a;              // ... and its record
    auto fetch_record = [&](int idx) {
      if (idx < p.n_prefill_items) {
        rec_a = __ldg(reinterpret_cast<const int4*>(p.prefill_items) + 2 * idx);
        rec_b = __ldg(reinterpret_cast<const int4*>(p.prefill_items) + 2 * idx + 1);
      }
    };
    if (pi == 0 && lane == 0) fetch_record(q_next);
    for (;;) {
      int item = 0;
      bool ok = true;
      ItemView v{};
      if (pi == 0) {
        if (lane == 0) {
          ok = mbar_wait(&bar->ring_empty[rs], rph ^ 1, abort_flag, p.status);
          if (ok) {
            item = q_next;
            if (item < p.n_prefill_items) v = view_item(p, rec_a, rec_b, Mt);
            bar->ring_item[rs] = item;
            bar->ring_view[rs] = v;
            mbar_arrive(&bar->ring_full[rs]);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        __syncwarp();
        item = bar->ring_item[rs];
        v = bar->ring_view[rs];
      } else {
        ok = mbar_wait(&bar->ring_full[rs], rph, abort_flag, p.status);
        if (!__all_sync(0xffffffffu, ok)) break;
        item = bar->ring_item[rs];
        v = bar->ring_view[rs];
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar->ring_empty[rs]);
      }
      if (++rs == 2) { rs = 0; rph ^= 1; }
      if (item >= p.n_prefill_items) break;
      const int32_t* table = p.block_tables + size_t(v.seq) * p.max_pages_per_seq;
      const int n_pages = (v.n_keys + 15) >> 4;
      int pg_next = lane < n_pages ? table[lane] : 0, pg_cur = 0;
      {
        // Q tiles: one box of Mt token rows x 64 columns per (tile, head, half) -- up to 32 copies per item, which one
        // thread would need microseconds to issue.  The four producers take every fourth copy each, one lane per copy.
        if (lane == 0) ok = mbar_wait(&bar->q_empty, (n_items_seen & 1) ^ 1, abort_flag, p.status);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (ok) {
          const int n_tiles = v.n_tok_t[1] > 0 ? 2 : 1;
          const int n_copies = n_tiles * G * G_::HALVES;
          if (pi == 0 && lane == 0) mbar_expect_tx(&bar->q_full, n_copies * Mt * 128);
          const int cidx = pi + 4 * lane;                    // copy of this lane: (tile, head, half), half fastest
          if (cidx < n_copies) {
            const int h = cidx % G_::HALVES, g = (cidx / G_::HALVES) % G, t = cidx / (G_::HALVES * G);
            tma_load_2d(q_smem + t * G_::Q_BYTES + h * 16384 + g * Mt * 128, &p.tm_q, &bar->q_full,
                        (v.hk * G + g) * DH + h * 64, v.tok0 + t * Mt);
          }
        }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      ++n_items_seen;
      for (int kb = 0; kb < v.nblk && ok; ++kb) {
        if (pi == 0 && lane == 0) {
          if (kb == max(0, v.nblk - 4)) q_next = int(gridDim.x) + atomicAdd(p.counters, 1);
          if (kb == v.nblk - 2 && v.nblk > 2) fetch_record(q_next);
        }
        if ((kb & 7) == 0) {
          pg_cur = pg_next;
          const int idx = (kb + 8) * 4 + lane;
          pg_next = idx < n_pages ? table[idx] : 0;
        }
        const uint32_t gb = blk_base + kb;
        const int rem = v.n_keys - kb * PF_KEYS;
        const int np = rem >= PF_KEYS ? 4 : (rem + 15) >> 4;        // pages of the block that exist
        const int mine = np - w0 >= 2 ? 2 : (np - w0 > 0 ? np - w0 : 0);
        const uint32_t st = gb % (kv ? PF_VSTAGES : PF_KSTAGES), ph = (gb / (kv ? PF_VSTAGES : PF_KSTAGES)) & 1;
        uint64_t* full = kv ? &bar->v_full[st] : &bar->k_full[st];
        uint8_t* dst = (kv ? v_smem : k_smem) + st * G_::KV_BYTES;
        if (lane == 0) {
          ok = mbar_wait(kv ? &bar->v_empty[st] : &bar->k_empty[st], ph ^ 1, abort_flag, p.status);
          if (ok) {
            if (mine > 0) mbar_expect_tx(full, mine * G_::HALVES * 2048);
            else mbar_arrive(full);                                  // nothing to fetch, but the block counts on two arrivals
          }
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        for (int w = w0; w < w0 + mine; ++w) {
          const int page = __shfl_sync(0xffffffffu, pg_cur, (kb & 7) * 4 + w);
          if (lane == 0) {
            const int row = pool_row(p, kv, page, v.hk);
            for (int h = 0; h < G_::HALVES; ++h) tma_load_2d(dst + h * 8192 + w * 2048, &p.tm_kv, full, h * 64, row);
          }
        }
      }
      if (!ok) break;
      if (pi == 0 && lane == 0 && v.nblk <= 2) fetch_record(q_next);   // (a short item: not before its own requests are out)
      blk_base += v.nblk;
    }
  } else if (warp == 9 || warp == 10) {
    // ============================================================ MMA issuers ==
    // One issuing thread per tile (warp 9: tile A, warp 10: tile B).  Every wait and every commit costs its thread
    // on the order of a hundred cycles even when nothing has to be waited for; with a thread per tile those sit
    // beside the other tile's MMAs instead of between them (the tensor core takes the instructions of both threads
    // in the order they arrive; each thread's own order is all that the overlay of P on S relies on).
    // The K and V slots and the Q tiles are released by both threads (barriers of two arrivals): a thread with
    // no block to compute -- its tile is absent or shorter -- arrives without a commit, but only after it has seen
    // the slot filled, so that its arrival cannot fall into an earlier phase of the barrier.
    if (lane == 0) {
      const int t = warp - 9;
      constexpr uint32_t idesc_s = umma_idesc_bf16_f32(128, PF_KEYS);
      constexpr uint32_t idesc_pv = umma_idesc_bf16_f32(128, DH) | (1u << 16);   // B (= V) is MN-major
      // descriptors of this tile's Q / the first K slot / the first V slot (shared memory is below 256 KB, so adding
      // byte offsets / 16 to a descriptor never carries out of its address field)
      const uint64_t q_desc = umma_desc_kmajor_sw128(smem_u32(q_smem) + t * G_::Q_BYTES);
      const uint64_t k_desc0 = umma_desc_kmajor_sw128(smem_u32(k_smem));
      const uint64_t v_desc0 = umma_desc_mnmajor_sw128(smem_u32(v_smem), 8192, 1024);
      const uint32_t d_o = tmem + G_::O0 + t * DH, s_base = tmem + G_::S0 + t * 128;
      uint32_t g_s = 0, g_pv = 0;        // blocks of this tile whose S / whose P V has been issued, over all items
      bool ok = true;
      // O (+)= P(buffer) * V(block gb) for block j of the item, then the V slot goes back to the producer
      auto pv_block = [&](const ItemView& v, int j) -> bool {
        const uint32_t gb = blk_base + j, vst = gb % PF_VSTAGES;
        if (!mbar_wait(&bar->v_full[vst], (gb / PF_VSTAGES) & 1, abort_flag, p.status)) return false;
        if (j >= v.nblk_t[t]) {                                     // nothing of this tile in the block
          mbar_arrive(&bar->v_empty[vst]);
          return true;
        }
        const uint32_t buf = g_pv & 1, bph = (g_pv >> 1) & 1;
        if (!mbar_wait(&bar->p_full[t][buf], bph, abort_flag, p.status)) return false;
        tc_fence_after_sync();
        const uint64_t vdesc = v_desc0 + uint64_t(vst * (G_::KV_BYTES >> 4));
        const uint32_t a_p = s_base + buf * PF_KEYS, acc0 = j == 0 ? 0u : 1u;    // the item's first block overwrites O
#pragma unroll
        for (int pg = 0; pg < 4; ++pg)        // 16 keys (one page) per MMA: 8 columns of P
          umma_bf16_ts(d_o, a_p + 8 * pg, vdesc + uint64_t(pg * (2048 >> 4)), idesc_pv, pg != 0 ? 1u : acc0);
        // "P V of block c has completed" alternates between two barriers: a waiter that does not look at every block
        // is then never more than one phase of a barrier away from it (the scores of block c + 2, which it waits for
        // first, complete after the product of block c), so a parity wait cannot mistake one phase for another
        umma_commit(&bar->o_full[t][buf]);
        umma_commit(&bar->v_empty[vst]);
        ++g_pv;
        return true;
      };
      for (;;) {
        if (!mbar_wait(&bar->ring_full[rs], rph, abort_flag, p.status)) break;
        const int item = bar->ring_item[rs];
        const ItemView v = bar->ring_view[rs];
        mbar_arrive(&bar->ring_empty[rs]);
        if (++rs == 2) { rs = 0; rph ^= 1; }
        if (item >= p.n_prefill_items) break;
        const int nblk = v.nblk_t[t];
        if (!mbar_wait(&bar->q_full, n_items_seen & 1, abort_flag, p.status)) break;
        ++n_items_seen;
        if (nblk == 0) mbar_arrive(&bar->q_empty);
        for (int j = 0; j < v.nblk && ok; ++j) {
          const uint32_t gb = blk_base + j, kst = gb % PF_KSTAGES;
          if (!mbar_wait(&bar->k_full[kst], (gb / PF_KSTAGES) & 1, abort_flag, p.status)) { ok = false; break; }
          if (j < nblk) {
            tc_fence_after_sync();
            // the buffer held S and then P of block j - 2, whose P V product this thread issued in the previous round
            const uint32_t buf = g_s & 1;
            const uint64_t kdesc = k_desc0 + uint64_t(kst * (G_::KV_BYTES >> 4));
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks)
              umma_bf16(s_base + buf * PF_KEYS, q_desc + uint64_t((ks >> 2) * (16384 >> 4) + 2 * (ks & 3)),
                        kdesc + uint64_t((ks >> 2) * (8192 >> 4) + 2 * (ks & 3)), idesc_s, ks != 0);
            umma_commit(&bar->s_full[t][buf]);
            umma_commit(&bar->k_empty[kst]);                        // the K slot, once these scores are computed
            if (j == nblk - 1) umma_commit(&bar->q_empty);          // and the Q tile after the tile's last scores
            ++g_s;
          } else {
            mbar_arrive(&bar->k_empty[kst]);
          }
          if (j > 0) ok = pv_block(v, j - 1);                       // overlaps the softmax of block j
        }
        if (!ok || !pv_block(v, v.nblk - 1)) break;
        blk_base += v.nblk;
      }
    }
  } else {
    // ================================================================ softmax ==
    const int t = warp >> 2;                      // tile of this warp group
    const int r = threadIdx.x & 127;              // row of the tile = TMEM lane
    const uint32_t lane_base = uint32_t((warp & 3) * 32) << 16;
    const uint32_t s_col = G_::S0 + t * 128, o_col = G_::O0 + t * DH;
    uint32_t g = 0;                               // blocks this tile has processed, over all items
    for (;;) {
      bool ok = mbar_wait(&bar->ring_full[rs], rph, abort_flag, p.status);
      if (!__all_sync(0xffffffffu, ok)) break;
      const int item = bar->ring_item[rs];
      const ItemView v = bar->ring_view[rs];
      __syncwarp();
      if (lane == 0) mbar_arrive(&bar->ring_empty[rs]);
      if (++rs == 2) { rs = 0; rph ^= 1; }
      if (item >= p.n_prefill_items) break;
      const int nblk = v.nblk_t[t], n_tok = v.n_tok_t[t];
      if (nblk == 0) { blk_base += v.nblk; continue; }            // the item has no tile for this warp group
      const int hg = r / Mt, tok = r - hg * Mt;
      const bool row_valid = hg < G && tok < n_tok;
      // last key a row sees: its own position (padding rows behave like the tile's last token), or the sequence's last key
      const int pos = p.bidirectional ? v.n_keys - 1 : v.pos0 + t * Mt + min(tok, n_tok - 1);

      float m_ref = -INFINITY, l_run = 0.f;
      uint32_t sreg[32], sreg2[32];
      for (int j = 0; j < nblk; ++j, ++g) {
        const uint32_t buf = g & 1, bph = (g >> 1) & 1;
        ok = mbar_wait(&bar->s_full[t][buf], bph, abort_flag, p.status);
        if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
        tc_fence_after_sync();
        const int key0 = j * PF_KEYS;
        tmem_ld32(tmem + lane_base + s_col + buf * PF_KEYS, sreg);
        tmem_ld32(tmem + lane_base + s_col + buf * PF_KEYS + 32, sreg2);
        tmem_ld_wait();
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
        // the reference maximum (kept on the raw scores; the 1/sqrt(Dh) * log2(e) scale is folded into the
        // exponent) moves only when the block's maximum is far above it
        float alpha = 1.f;
        const bool move = row_valid && (j == 0 || (mx - m_ref) * scale_log2 > kRefSlack);
        if (j == 0) m_ref = mx;
        else if (move) {
          alpha = fast_exp2((m_ref - mx) * scale_log2);
          m_ref = mx;
        }
        const bool rescale = j > 0 && __any_sync(0xffffffffu, move);
        const float neg_ms = -m_ref * scale_log2;
        float sum = 0.f;
        uint32_t pk[32];
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          const float a0 = fast_exp2(fmaf(__uint_as_float(sreg[e]), scale_log2, neg_ms));
          const float a1 = fast_exp2(fmaf(__uint_as_float(sreg[e + 1]), scale_log2, neg_ms));
          const float b0 = fast_exp2(fmaf(__uint_as_float(sreg2[e]), scale_log2, neg_ms));
          const float b1 = fast_exp2(fmaf(__uint_as_float(sreg2[e + 1]), scale_log2, neg_ms));
          sum += (a0 + a1) + (b0 + b1);
          pk[e >> 1] = pack_bf16(a0, a1);
          pk[16 + (e >> 1)] = pack_bf16(b0, b1);
        }
        l_run = l_run * alpha + sum;
        if (rescale) {
          // O must be at rest: the P V product of the previous block has completed (its successor cannot be issued
          // before this warp group hands over P)
          ok = mbar_wait(&bar->o_full[t][(g - 1) & 1], ((g - 1) >> 1) & 1, abort_flag, p.status);
          if (!__all_sync(0xffffffffu, ok)) { ok = false; break; }
          tc_fence_after_sync();
#pragma unroll
          for (int c = 0; c < DH / 32; ++c) {
            tmem_ld32(tmem + lane_base + o_col + c * 32, sreg);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) sreg[e] = __float_as_uint(__uint_as_float(sreg[e]) * alpha);
            tmem_st32(tmem + lane_base + o_col + c * 32, sreg);
          }
          tmem_st_wait();
        }
        // P over the first 32 columns of the S buffer just read: column c of row r = keys 2 c, 2 c + 1
        tmem_st32(tmem + lane_base + s_col + buf * PF_KEYS, pk);
        // ragged last block of the item: V rows of keys that do not exist must not carry stray NaN / Inf bits
        const int n_valid = v.n_keys - key0;
        if (n_valid < PF_KEYS) {
          const uint32_t gb = blk_base + j, s = gb % PF_VSTAGES;
          const bool w = mbar_wait(&bar->v_full[s], (gb / PF_VSTAGES) & 1, abort_flag, p.status);
          if (!__all_sync(0xffffffffu, w)) { ok = false; break; }
          uint8_t* vst = v_smem + s * G_::KV_BYTES;
          const int n_units = (PF_KEYS - n_valid) * G_::HALVES * 8;
          for (int idx = r; idx < n_units; idx += 128) {
            const int u = idx & 7, h = (idx >> 3) % G_::HALVES, k = n_valid + (idx >> 3) / G_::HALVES;
            *reinterpret_cast<uint4*>(vst + h * 8192 + (k >> 4) * 2048 + (k & 15) * 128 + (u << 4)) =
                make_uint4(0, 0, 0, 0);
          }
          fence_proxy_async();
        }
        tmem_st_wait();
        tc_fence_before_sync();
        mbar_arrive(&bar->p_full[t][buf]);
      }
      if (!ok) break;
      // the item's last P V product, then the tile's rows of O leave through registers
      ok = mbar_wait(&bar->o_full[t][(g - 1) & 1], ((g - 1) >> 1) & 1, abort_flag, p.status);
      if (!__all_sync(0xffffffffu, ok)) break;
      tc_fence_after_sync();
      const float inv = 1.f / l_run;
      const bool f16 = p.o_f16 != 0;
      __nv_bfloat16* dst = p.o + size_t(v.tok0 + t * Mt + tok) * q_dim + (v.hk * G + hg) * DH;
#pragma unroll
      for (int c = 0; c < DH / 32; ++c) {
        tmem_ld32(tmem + lane_base + o_col + c * 32, sreg);
        tmem_ld_wait();
        if (row_valid) {
          float o32[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) o32[e] = __uint_as_float(sreg[e]) * inv;
          if (f16) note_f16_saturation(o32, p.status);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            uint4 w;
            w.x = pack_act(o32[u * 8 + 0], o32[u * 8 + 1], f16);
            w.y = pack_act(o32[u * 8 + 2], o32[u * 8 + 3], f16);
            w.z = pack_act(o32[u * 8 + 4], o32[u * 8 + 5], f16);
            w.w = pack_act(o32[u * 8 + 6], o32[u * 8 + 7], f16);
            *reinterpret_cast<uint4*>(dst + c * 32 + u * 8) = w;
          }
        }
      }
      tc_fence_before_sync();
      blk_base += v.nblk;
    }
  }

  // --------------------------------------------------------------- teardown --
  __syncwarp();
  if (*abort_flag) drain_after_abort();
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 9) {
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
