// Persistent, SM-budgeted bf16 GEMM on the 5th-generation tensor cores (tcgen05) with the step's
// element-wise work fused into its epilogues.
//
//   tile        pair kernel (more than 128 tokens): 256 x 256 per PAIR of blocks (a cluster of two SMs,
//               tcgen05.mma.cta_group::2): each block stages its 128 token rows of A and ONE 128-row half
//               of B per 64-wide K block (32 KB, 6-stage ring), the leader block issues M256 N256 K16 MMAs
//               that read both blocks' shared memory, and each block owns the accumulator rows of its
//               SM's tensor memory.  Halving the B bytes per SM is what lifts the operand-feed limit of the
//               single-block kernel (128 x 256 tile, 48 KB per K block, 4-stage ring), which remains for
//               small token counts, for sm_budget 1 and for the K-split path; both produce the same bits.
//   operands    TMA (128-byte swizzle) -> shared-memory ring -> tcgen05.mma, fp32 accumulators in tensor
//               memory, two accumulator buffers so the epilogue of tile i overlaps the main loop of i+1
//   roles       warp 0: TMA producer, warp 1: MMA issuer (one thread, leader block only), warps 2..5:
//               epilogue.  Cross-block signalling in a pair: both blocks' TMA bytes are counted on the
//               leader's "full" barrier; the leader's tcgen05.commit arrives on the "empty" and
//               "accumulator full" barriers of both blocks; epilogue warps of both blocks arrive on the
//               leader's "accumulator empty" barrier.
//   schedule    unit = worker + i * workers, workers <= sm_budget (pairs: sm_budget / 2), one block per
//               SM.  Each output tile is produced by one block (pair) with a fixed K order, so results do
//               not depend on the budget.
//
// Epilogues: residual add (the fp32 tile is ADDED into the residual stream by a TMA reduction, so the
// stream is never read by the SM), QKV (rotate-half RoPE; bf16 q by TMA store; k, v scattered into the
// paged cache), gate/up (silu(gate) * up -> bf16 by TMA store).  Output blocks are staged in shared memory
// in the 128-byte-swizzled layout the tensor maps expect (conflict-free for one-row-per-thread writes).
#include "kernels.h"
#include "ptx.cuh"

namespace hs {
namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int A_BYTES = BM * BK * 2;            // 16 KB
constexpr int BH_BYTES = 128 * BK * 2;          // one 128-row half of the B tile, 16 KB
// One block per tile: a stage holds A and both halves of B, 4 stages.  Block pair per 256 x 256 tile: every
// block stages A and ONE half of B (the MMA reads the other half from the other block), 6 stages.
template <bool PAIR> struct Ring {
  static constexpr int STAGE_BYTES = PAIR ? A_BYTES + BH_BYTES : A_BYTES + 2 * BH_BYTES;
  static constexpr int STAGES = PAIR ? 6 : 4;
};
constexpr int RING_BYTES = 4 * (A_BYTES + 2 * BH_BYTES);
static_assert(Ring<true>::STAGES * Ring<true>::STAGE_BYTES == RING_BYTES, "both rings fill the same space");
constexpr int kMaxStages = 12;                  // barrier slots; the ring holds fewer when stages are large
constexpr int GEMM_THREADS = 192;
constexpr int TMEM_COLS = 512;                  // two 128 x 256 fp32 accumulators
constexpr int EPI_BUF_BYTES = 4096;             // 32 rows x 128 B: a 32 x 32 fp32 or 32 x 64 bf16 output block
constexpr int EPI_WARP_BYTES = 2 * EPI_BUF_BYTES;   // two blocks per epilogue warp, filled alternately
constexpr int GEMM_SMEM = 1024 + RING_BYTES + 4 * EPI_WARP_BYTES + 384;
static_assert(GEMM_SMEM <= 227 * 1024, "fits one SM");
static_assert(GEMM_SMEM >= kMinSmemBytes, "one block per SM");

// Qkv mode, single blocks: tiles of 128 virtual columns (one B box) when p.bn says so -- the launcher asks for
// them at small M, where the tile count decides how many SMs stream weights; 256 otherwise.  A 128-column
// tile never straddles q | k | v (their widths are multiples of 128) and holds whole heads.
__host__ __device__ __forceinline__ int gemm_qkv_width(const GemmParams& p) { return p.bn == 128 && !p.pair ? 128 : BN; }

// Output-tile width: 256 virtual columns, except in Resid mode where the launcher picks p.bn (a multiple
// of 32 in [128, 256]) from the problem shape so that the tile count fills whole waves of SMs.
__host__ __device__ __forceinline__ int gemm_n_tiles(const GemmParams& p) {
  if (p.mode == kGemmGateUp) return (p.N + 127) / 128;
  const int bn = p.mode == kGemmResid ? p.bn : gemm_qkv_width(p);
  return (p.N + bn - 1) / bn;
}

struct BSource { int map, row; };
__device__ __forceinline__ BSource b_source(const GemmParams& p, int n_tile, int half) {
  if (p.mode == kGemmResid) return {0, n_tile * p.bn + half * 128};
  if (p.mode == kGemmGateUp) return {half, n_tile * 128};
  int v = n_tile * gemm_qkv_width(p) + half * 128;
  if (v < p.q_dim) return {0, v};
  v -= p.q_dim;
  if (v < p.kv_dim) return {1, v};
  return {2, v - p.kv_dim};
}

__device__ __forceinline__ float4 ld4(const float* p) { return *reinterpret_cast<const float4*>(p); }

__device__ __forceinline__ void store_bf16x32(__nv_bfloat16* dst, const float (&v)[32], int n_valid) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (i * 8 < n_valid) {
      uint4 w;
      w.x = pack_bf16(v[i * 8 + 0], v[i * 8 + 1]);
      w.y = pack_bf16(v[i * 8 + 2], v[i * 8 + 3]);
      w.z = pack_bf16(v[i * 8 + 4], v[i * 8 + 5]);
      w.w = pack_bf16(v[i * 8 + 6], v[i * 8 + 7]);
      *reinterpret_cast<uint4*>(dst + i * 8) = w;
    }
  }
}

// Staging layout of an output block: row r (one thread of the warp) is 128 bytes = 8 units of 16 B,
// unit u stored at r * 128 + ((u ^ (r & 7)) << 4): the 128-byte swizzle of the output tensor maps.
__device__ __forceinline__ void stage_f32x32(uint8_t* buf, int lane, const uint32_t (&r)[32]) {
#pragma unroll
  for (int u = 0; u < 8; ++u)
    *reinterpret_cast<uint4*>(buf + lane * 128 + ((u ^ (lane & 7)) << 4)) =
        make_uint4(r[4 * u], r[4 * u + 1], r[4 * u + 2], r[4 * u + 3]);
}
// 32 values -> bf16 into units u0 .. u0+3 of the thread's row (u0 = 0 or 4: which 32 of the 64 columns).
__device__ __forceinline__ void stage_bf16x32(uint8_t* buf, int lane, int u0, const float (&v)[32], bool f16 = false) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    uint4 w;
    w.x = pack_act(v[i * 8 + 0], v[i * 8 + 1], f16);
    w.y = pack_act(v[i * 8 + 2], v[i * 8 + 3], f16);
    w.z = pack_act(v[i * 8 + 4], v[i * 8 + 5], f16);
    w.w = pack_act(v[i * 8 + 6], v[i * 8 + 7], f16);
    *reinterpret_cast<uint4*>(buf + lane * 128 + (((u0 + i) ^ (lane & 7)) << 4)) = w;
  }
}

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Bounded spin on a global word written by another block (same limits as the mbarrier waits).
__device__ __forceinline__ bool spin_until_equal(const int* word, int value, volatile int* abort_flag, int* status) {
  const unsigned long long t0 = globaltimer_ns();
  for (uint32_t spins = 0;; ++spins) {
    if (ld_acquire(word) == value) return true;
    if ((spins & 0x3f) == 0x3f) {
      if (*abort_flag) return false;
      if (globaltimer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(status, kErrTimeout);
        return false;
      }
      __nanosleep(100);
    }
  }
}

// r[0..31] += b[0..31]: fp32 values held as raw bits, bias in bf16 (64-byte aligned; the same for every row,
// so the loads of a warp are broadcasts out of the L1).
__device__ __forceinline__ void add_bias32(uint32_t (&r)[32], const __nv_bfloat16* b) {
  const uint4* src = reinterpret_cast<const uint4*>(b);
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const uint4 w = __ldg(src + u);
    const uint32_t pk[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      r[u * 8 + 2 * e] = __float_as_uint(__uint_as_float(r[u * 8 + 2 * e]) + __uint_as_float(pk[e] << 16));
      r[u * 8 + 2 * e + 1] = __float_as_uint(__uint_as_float(r[u * 8 + 2 * e + 1]) + __uint_as_float(pk[e] & 0xffff0000u));
    }
  }
}

// r[0..31] *= s (fp32 values held as raw bits)
__device__ __forceinline__ void scale32(uint32_t (&r)[32], float s) {
#pragma unroll
  for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * s);
}

// Folded RMSNorm, producing side: a thread leaves the sum of x^2 of its row over one tile column; the warp that
// delivers the last tile column of its 32 rows (counted per row group) adds each row's partials in tile-column order --
// the same sum whoever comes last -- and writes r = rsqrt(mean(x^2) + eps) for the GEMM that follows.
__device__ __forceinline__ void finish_row_norm(const GemmParams& p, int row, bool row_ok, int row_group, int n,
                                                int n_n_tiles, float ss, int lane) {
  if (row_ok) p.row_ss[size_t(row) * p.ss_stride + n] = ss;
  __threadfence();
  __syncwarp();
  int last = 0;
  if (lane == 0) last = atomicAdd(p.row_group_done + row_group, 1) == n_n_tiles - 1;
  last = __shfl_sync(0xffffffffu, last, 0);
  if (!last) return;
  __threadfence();
  if (row_ok) {
    float sum = 0.f;
    for (int i = 0; i < n_n_tiles; ++i) sum += __ldcg(p.row_ss + size_t(row) * p.ss_stride + i);
    p.row_rs[row] = rsqrtf(sum / float(p.N) + p.norm_eps);
  }
  if (lane == 0) p.row_group_done[row_group] = 0;      // ready for the next launch
}

// Address of element e of (slot, kv head) in one layer's K or V pages.
__device__ __forceinline__ __nv_bfloat16* cache_ptr(__nv_bfloat16* base, int slot, int hk, int n_kv_heads, int Dh,
                                                    int e) {
  const size_t row = (size_t(slot >> 4) * n_kv_heads + hk) * 16 + (slot & 15);
  return base + row * Dh + e;
}

// One work unit of a block (pair): the K blocks [kb_begin, kb_end) of an output tile.  `seg` counts the earlier K
// segments of the same tile (their sums are added into the output before this one's), `last` marks the tile's final
// segment.
struct Unit { int tile, kb_begin, kb_end, seg, last, half; };

// Hands a worker its units, in the same order for the producer, the MMA issuer and the epilogue warps.
//   plain / split-K   unit u = worker + i * workers over tiles x splits, split-major (a split's predecessors have
//                     smaller unit numbers).
//   stream-K          (Resid mode on pairs, chosen by shape) the tiles' K blocks, laid end to end tile after tile, are
//                     cut into `n_slots` equal runs -- one per pair of the whole device, whatever the budget -- so that
//                     no pair idles through a ragged last wave.  A run is a tail segment of one tile, whole tiles, and
//                     a head segment of another; slot s is worked by worker s mod workers.  Within a slot the head
//                     segment comes first and the tail segment last: the tail's predecessor is the head segment of
//                     the previous slot, which that slot has done first, so the ordered add never waits long.
//                     With sm_budget 1 there is no pair: the single block then works the same slots on the same
//                     256-row tiles, each unit twice -- once per 128-row half (`half`) -- so that every output
//                     element still receives the same partial sums in the same order.
struct UnitWalk {
  int stream_k, n_tiles, k_blocks, ksplit, n_workers, n_slots;
  int halves, n_m_tiles, M;  // halves = 2: a single block standing in for a pair
  int cur;                 // unit (plain) or slot (stream-K) being handed out
  int idx, n_seg, first_tile;
  long long lo, hi;
  __device__ __forceinline__ void init(const GemmParams& p, bool pair, bool emulate_pair, int n_m_tiles_, int n_tiles_,
                                       int k_blocks_, int worker, int n_workers_) {
    stream_k = (pair || emulate_pair) && p.mode == kGemmResid && p.stream_k_slots > 0;
    halves = emulate_pair ? 2 : 1;
    n_m_tiles = n_m_tiles_;
    M = p.M;
    n_tiles = n_tiles_; k_blocks = k_blocks_; n_workers = n_workers_;
    ksplit = !pair && p.mode == kGemmResid && p.ksplit > 1 ? p.ksplit : 1;
    n_slots = stream_k ? p.stream_k_slots : n_tiles * ksplit;
    cur = worker - n_workers;
    idx = n_seg = 0; first_tile = 0; lo = hi = 0;
  }
  __device__ __forceinline__ bool next(Unit& u) {
    if (halves == 2 && idx > 0 && u.half == 0) {   // the second half of the unit handed out last, if it has rows
      if ((2 * (u.tile % n_m_tiles) + 1) * BM < M) {
        u.half = 1;
        return true;
      }
    }
    u.half = 0;
    if (!stream_k) {
      cur += n_workers;
      if (cur >= n_slots) return false;
      const int ks = cur / n_tiles;
      u.tile = cur - ks * n_tiles;
      u.kb_begin = gemm_split_begin(k_blocks, ksplit, ks);
      u.kb_end = gemm_split_begin(k_blocks, ksplit, ks + 1);
      u.seg = ks;
      u.last = ks == ksplit - 1;
      return true;
    }
    const long long total = (long long)n_tiles * k_blocks;
    while (idx == n_seg) {                         // next slot of this worker (empty slots are skipped)
      cur += n_workers;
      if (cur >= n_slots) return false;
      lo = total * cur / n_slots;
      hi = total * (cur + 1) / n_slots;
      idx = 0;
      n_seg = 0;
      if (hi > lo) {
        first_tile = int(lo / k_blocks);
        n_seg = int((hi - 1) / k_blocks) - first_tile + 1;
      }
    }
    const int nat = n_seg == 1 ? 0 : (idx == 0 ? n_seg - 1 : (idx == n_seg - 1 ? 0 : idx));
    const int t = first_tile + nat;
    const long long t0 = (long long)t * k_blocks;
    const long long b = lo > t0 ? lo : t0, e = hi < t0 + k_blocks ? hi : t0 + k_blocks;
    u.tile = t;
    u.kb_begin = int(b - t0);
    u.kb_end = int(e - t0);
    // earlier segments of the tile = slot boundaries inside the tile before this segment; the slot that holds the
    // tile's first K block is ceil((t0 + 1) n_slots / total) - 1
    u.seg = u.kb_begin == 0 ? 0 : cur - (int(((t0 + 1) * n_slots + total - 1) / total) - 1);
    u.last = u.kb_end == k_blocks;
    ++idx;
    return true;
  }
};

template <bool PAIR>
__device__ __forceinline__ void gemm_body(const GemmParams& p) {
  // Ring geometry.  Pairs: 6 stages of 32 KB.  Single blocks: a stage holds the A box (128 rows, or only 64 / 32
  // when the step is that small) and one or two 128-row B boxes, and the ring holds as many stages as fit (at
  // most kMaxStages): a block's streaming rate is stages in flight / memory latency, so the small stages of a
  // small step buy depth -- 8 or 9 stages instead of 4.
  const bool b_two = p.mode == kGemmGateUp || (p.mode == kGemmResid ? p.bn : gemm_qkv_width(p)) > 128;
  const int a_bytes = (p.a_box_rows > 0 && !PAIR ? p.a_box_rows : BM) * BK * 2;
  const int STAGE_BYTES = PAIR ? Ring<true>::STAGE_BYTES : a_bytes + (b_two ? 2 : 1) * BH_BYTES;
  // (a pair kernel that folds the following RMSNorm into its epilogue runs its ring one stage short and uses the last
  // stage's 32 KB as landing blocks for the residual stream: see the epilogue)
  const bool fold_pair = PAIR && p.mode == kGemmResid && p.norm_gain != nullptr;
  const int STAGES = PAIR ? Ring<true>::STAGES - (fold_pair ? 1 : 0)
                          : (RING_BYTES / STAGE_BYTES < kMaxStages ? RING_BYTES / STAGE_BYTES : kMaxStages);
  const int b_off = PAIR ? A_BYTES : a_bytes;     // B boxes follow the A box inside a stage
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* epi_smem = smem + RING_BYTES;
  uint64_t* full = reinterpret_cast<uint64_t*>(epi_smem + 4 * EPI_WARP_BYTES);
  uint64_t* empty = full + kMaxStages;
  uint64_t* tfull = empty + kMaxStages;
  uint64_t* tempty = tfull + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint64_t* xbar = reinterpret_cast<uint64_t*>(epi_smem + 4 * EPI_WARP_BYTES + 256);   // [4 warps][4] landing-block barriers (three used)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  log_smid(p.smid_log);
  // In pair mode the two blocks of a cluster share every work unit: a unit's tile is 256 rows tall and
  // block `rank` owns rows 128 * rank .. 128 * rank + 127 of it.
  const uint32_t rank = PAIR ? cluster_ctarank() : 0;
  const int worker = PAIR ? int(blockIdx.x >> 1) : int(blockIdx.x);
  const int n_workers = PAIR ? int(gridDim.x >> 1) : int(gridDim.x);
  // a single block that stands in for a pair (stream-K form at sm_budget 1) walks the pair's 256-row tiles
  const bool emulate_pair = !PAIR && p.pair && p.mode == kGemmResid && p.stream_k_slots > 0;
  const int n_m_tiles = PAIR || emulate_pair ? (p.M + 2 * BM - 1) / (2 * BM) : (p.M + BM - 1) / BM;
  const int n_n_tiles = gemm_n_tiles(p);
  const int n_tiles = n_m_tiles * n_n_tiles;
  const int k_blocks = (p.K + BK - 1) / BK;
  // Work unit = (output tile, run of K blocks): see UnitWalk.  Runs shorter than the whole K range exist only in
  // Resid mode, whose epilogue adds partial sums into the output in a fixed order.
  UnitWalk walk;
  walk.init(p, PAIR, emulate_pair, n_m_tiles, n_tiles, k_blocks, worker, n_workers);
  const bool ordered = walk.stream_k || walk.ksplit > 1;
  Unit un;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&tfull[i], 1);
      mbar_init(&tempty[i], PAIR ? 8 : 4);      // one arrival per epilogue warp (of both blocks)
    }
    for (int i = 0; i < 16; ++i) mbar_init(&xbar[i], 1);
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&p.tm_a);
    tma_prefetch_desc(&p.tm_b[0]);
    tma_prefetch_desc(p.mode == kGemmResid ? &p.tm_out : p.mode == kGemmQkv ? &p.tm_q : &p.tm_act);
  }
  if (warp == 1) {
    if (PAIR) {
      tmem_alloc_pair(tmem_slot, TMEM_COLS);
      tmem_relinquish_pair();
    } else {
      tmem_alloc(tmem_slot, TMEM_COLS);
      tmem_relinquish();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (PAIR) cluster_sync_all();               // the other block's barriers exist before anything targets them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // A small step's A box holds only the rows that exist (32 or 64 instead of 128): the MMA still reads 128
  // rows starting at the stage's base -- beyond the A box that is the B data of the stage, finite values
  // that only reach accumulator rows no epilogue stores
  const bool two_halves = b_two;
  // One stage's requests of the producer thread: the weight boxes (which also arm the barrier) and the A box.  In a
  // pair both blocks' bytes are counted on the leader's barrier, which the leader arms for both.
  auto load_b = [&](int s, int kb, const BSource& b0, const BSource& b1) {
    uint8_t* st = smem + s * STAGE_BYTES;
    if (PAIR) {
      if (rank == 0) mbar_expect_tx(&full[s], 2 * STAGE_BYTES);
      tma_load_2d_pair(st + b_off, &p.tm_b[b0.map], mapa_u32(smem_u32(&full[s]), 0), kb * BK, b0.row);
    } else {
      mbar_expect_tx(&full[s], a_bytes + (two_halves ? 2 * BH_BYTES : BH_BYTES));
      tma_load_2d(st + b_off, &p.tm_b[b0.map], &full[s], kb * BK, b0.row);
      if (two_halves) tma_load_2d(st + b_off + BH_BYTES, &p.tm_b[b1.map], &full[s], kb * BK, b1.row);
    }
  };
  auto load_a = [&](int s, int kb, int m, int half) {
    uint8_t* st = smem + s * STAGE_BYTES;
    if (PAIR) tma_load_2d_pair(st, &p.tm_a, mapa_u32(smem_u32(&full[s]), 0), kb * BK, (2 * m + int(rank)) * BM);
    else tma_load_2d(st, &p.tm_a, &full[s], kb * BK, (emulate_pair ? 2 * m + half : m) * BM);
  };
  // The weights never change: the producer asks for the weight boxes of its first unit's first stages before the wait
  // for the previous kernel, and for the A boxes of those stages after it.
  bool have_unit = false;
  int b_ahead = 0;
  if (warp == 0 && lane == 0) {
    have_unit = walk.next(un);
    if (have_unit) {
      const int n = un.tile / n_m_tiles;
      const BSource b0 = b_source(p, n, PAIR ? int(rank) : 0), b1 = b_source(p, n, 1);
      b_ahead = un.kb_end - un.kb_begin < STAGES ? un.kb_end - un.kb_begin : STAGES;
      for (int i = 0; i < b_ahead; ++i) load_b(i, un.kb_begin + i, b0, b1);
    }
  }
  griddep_wait();                 // everything above is set-up; the operands belong to the previous kernel until here
  griddep_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------- TMA producer --
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      while (ok && have_unit) {
        const int tile = un.tile;
        const int m = tile % n_m_tiles, n = tile / n_m_tiles;
        const BSource b0 = b_source(p, n, PAIR ? int(rank) : 0), b1 = b_source(p, n, 1);
        const int kb_end = un.kb_end;
        for (int kb = un.kb_begin; kb < kb_end; ++kb) {
          if (!mbar_wait(&empty[s], ph ^ 1, abort_flag, p.status)) { ok = false; break; }
          if (b_ahead > 0) --b_ahead;
          else load_b(s, kb, b0, b1);
          load_a(s, kb, m, un.half);
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
        have_unit = walk.next(un);
      }
    }
  } else if (warp == 1) {
    // --------------------------------------------------------- MMA issuer --
    if (lane == 0 && rank == 0) {
      // both operands are fp16 or both bf16 (one MMA cannot mix the two): the format fields of A (bits 7..9)
      // and B (bits 10..12) are 0 for fp16 and 1 for bf16
      const uint32_t idesc = umma_idesc_bf16_f32(PAIR ? 2 * BM : BM,
                                                 PAIR ? BN : p.mode == kGemmResid ? p.bn : p.mode == kGemmQkv ? gemm_qkv_width(p) : BN) &
                             (p.ab_f16 ? ~(63u << 7) : ~0u);
      int s = 0, acc = 0;
      uint32_t ph = 0, acc_ph = 0;
      bool ok = true;
      const uint64_t a_desc0 = umma_desc_kmajor_sw128(smem_u32(smem));
      while (ok && walk.next(un)) {
        if (!mbar_wait(&tempty[acc], acc_ph ^ 1, abort_flag, p.status)) break;
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        const int kb_begin = un.kb_begin, kb_end = un.kb_end;
        for (int kb = kb_begin; kb < kb_end; ++kb) {
          if (!mbar_wait(&full[s], ph, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after_sync();
          // descriptors of stage s: those of stage 0 plus the stage's offset in the address field (units of 16 bytes;
          // shared memory is below 256 KB, so nothing carries out of the field): the issuing thread has as little as
          // possible between two MMAs
          const uint64_t a_desc = a_desc0 + uint64_t(s * (STAGE_BYTES >> 4));
          const uint64_t b_desc = a_desc + uint64_t(b_off >> 4);
          const uint32_t acc0 = kb != kb_begin ? 1u : 0u;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {  // 16 bf16 = 32 B along K: +2 in the (address / 16) field
            if (PAIR) umma_bf16_pair(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, k != 0 ? 1u : acc0);
            else umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, k != 0 ? 1u : acc0);
          }
          // frees the stage (in both blocks) once these MMAs have read it
          if (PAIR) {
            umma_commit_pair_both(&empty[s]);
          } else {
            umma_commit(&empty[s]);
          }
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
        if (ok) {
          if (PAIR) {
            umma_commit_pair_both(&tfull[acc]);
          } else {
            umma_commit(&tfull[acc]);
          }
        }
        acc ^= 1;
        if (acc == 0) acc_ph ^= 1;
      }
    }
  } else {
    // ----------------------------------------------------------- epilogue --
    const int quarter = warp & 3;             // the TMEM lane quarter this warp may read
    int acc = 0;
    uint32_t acc_ph = 0;
    const int Dh = p.head_dim;
    uint8_t* epi_buf = epi_smem + quarter * EPI_WARP_BYTES;
    int epi_sel = 0;                          // staging block to fill next
    uint32_t xph = 0;                         // phase bits of this warp's landing-block barriers
    while (walk.next(un)) {
      const int tile = un.tile, ks = un.seg;
      const int m = PAIR ? 2 * (tile % n_m_tiles) + int(rank)
                         : emulate_pair ? 2 * (tile % n_m_tiles) + un.half : tile % n_m_tiles,
                n = tile / n_m_tiles;
      const int row = m * BM + quarter * 32 + lane;
      const bool row_ok = row < p.M;
      const int row_base = m * BM + quarter * 32;          // first row of this warp's 32
      // folded RMSNorm, consuming side: r of this thread's row, requested before the wait for the accumulator
      float rs = 1.f;
      if (p.in_row_rs != nullptr && p.mode != kGemmResid && row_ok) rs = __ldcg(p.in_row_rs + row);
      // folded RMSNorm, producing side: the first two blocks of this warp's rows of y are on their way before the
      // tile's products are complete
      const bool fold_now = fold_pair && un.last;
      // three landing blocks per warp: two in the ring's unused last stage, the third is the warp's second staging block
      uint8_t* xb_stage = smem + (Ring<true>::STAGES - 1) * Ring<true>::STAGE_BYTES + quarter * 2 * EPI_BUF_BYTES;
      auto landing = [&](int i) -> uint8_t* { return i < 2 ? xb_stage + i * EPI_BUF_BYTES : epi_buf + EPI_BUF_BYTES; };
      uint64_t* xb_bar = xbar + quarter * 4;
      const int n_chunks = min(p.bn / 32, (p.N - n * p.bn + 31) / 32);
      if (fold_now) {
        if (ordered && ks > 0) {              // every earlier segment of the tile must be in y before y is read
          int* turn = p.tile_turn + (tile * 2 + int(rank)) * 4 + quarter;
          bool go = true;
          if (lane == 0) go = spin_until_equal(turn, ks, abort_flag, p.status);
          if (!__shfl_sync(0xffffffffu, go, 0)) break;
        }
        if (lane == 0) {
          bulk_wait_read<0>();                // nothing of an earlier unit still reads the staging blocks
          for (int c = 0; c < 3 && c < n_chunks; ++c) {
            mbar_expect_tx(&xb_bar[c], EPI_BUF_BYTES);
            tma_load_2d(landing(c), &p.tm_out, &xb_bar[c], n * p.bn + c * 32, row_base);
          }
        }
      }
      const bool ok = mbar_wait(&tfull[acc], acc_ph, abort_flag, p.status);
      if (!__all_sync(0xffffffffu, ok)) break;
      tc_fence_after_sync();
      const uint32_t taddr = tmem_base + acc * BN + (uint32_t(quarter * 32) << 16);
      uint32_t r0[32], r1[32];
      float v0[32], v1[32];


      if (p.mode == kGemmResid) {
        // Ordered split-K: the partial sums of a tile are added into the output in split order, so the
        // result is the same fixed sum whatever block computed which split.  This warp owns 32 rows of the
        // tile; it waits until the previous split's add of those rows has been performed.
        int* turn = p.tile_turn + (PAIR ? tile * 2 + int(rank) : emulate_pair ? tile * 2 + un.half : tile) * 4 + quarter;
        if (ordered && ks > 0 && !fold_now) {
          bool go = true;
          if (lane == 0) go = spin_until_equal(turn, ks, abort_flag, p.status);
          if (!__shfl_sync(0xffffffffu, go, 0)) break;
        }
        const bool add = p.accumulate || ks > 0;
        // conditioned block: the product is scaled by the gate vector of the row's sequence before it is added
        const float* gate = p.gate_mod && row_ok ? p.gate_mod + (size_t(p.tok_seq[row]) * 6 + p.gate_which) * p.N : nullptr;
        if (gate) {   // pull this tile's part of the gate vector into the L1 before the chunk loop needs it
          const int chunk = lane % (p.bn / 32), col = n * p.bn + chunk * 32;
          if (col < p.N) asm volatile("prefetch.global.L1 [%0];" ::"l"(gate + col));
        }
        if (fold_now) {
          // Final segment of the tile with the following RMSNorm folded in: x = y + acc is formed here (every
          // earlier segment has been added into y), written back, and reused for h = 16-bit(x o g) and sum x^2.
          // The 32 x 32 blocks of y come in by TMA, one chunk ahead, into two landing blocks per warp (the ring's
          // unused last stage), are updated in place and leave by TMA stores; the 16-bit block of a pair of chunks
          // is staged beside them.
          const bool h16 = p.norm_h_f16 != 0;
          float ss = 0.f;
          uint8_t* buf_h = epi_buf;
          bool okx = true;
          for (int c = 0; c < n_chunks; ++c) {
            const int col0 = n * p.bn + c * 32;
            const int xi = c % 3;
            uint8_t* bx = landing(xi);
            if (lane == 0 && c > 0) {
              bulk_wait_read<0>();                         // the stores of the previous chunk have read their blocks
              if (c + 2 < n_chunks) {                      // ... so its landing block can take the chunk two further on
                const int xn = (c + 2) % 3;
                mbar_expect_tx(&xb_bar[xn], EPI_BUF_BYTES);
                tma_load_2d(landing(xn), &p.tm_out, &xb_bar[xn], col0 + 64, row_base);
              }
            }
            tmem_ld32(taddr + c * 32, r0);
            uint4 gw[4];                               // 32 gains (bf16), the same for every row
            const int nv = p.N - col0 >= 32 ? 8 : (p.N - col0) >> 2;
#pragma unroll
            for (int e = 0; e < 4; ++e)
              gw[e] = 2 * e < nv ? __ldg(reinterpret_cast<const uint4*>(p.norm_gain + col0) + e) : make_uint4(0, 0, 0, 0);
            okx = mbar_wait(&xb_bar[xi], (xph >> xi) & 1, abort_flag, p.status);
            if (!__all_sync(0xffffffffu, okx)) { okx = false; break; }
            xph ^= 1u << xi;
            tmem_ld_wait();
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              float4* slot = reinterpret_cast<float4*>(bx + lane * 128 + ((u ^ (lane & 7)) << 4));
              const float4 y4 = *slot;
              const float x0 = __uint_as_float(r0[4 * u]) + y4.x, x1 = __uint_as_float(r0[4 * u + 1]) + y4.y;
              const float x2 = __uint_as_float(r0[4 * u + 2]) + y4.z, x3 = __uint_as_float(r0[4 * u + 3]) + y4.w;
              if (u < nv) ss += (x0 * x0 + x1 * x1) + (x2 * x2 + x3 * x3);
              *slot = make_float4(x0, x1, x2, x3);
              r0[4 * u] = __float_as_uint(x0); r0[4 * u + 1] = __float_as_uint(x1);
              r0[4 * u + 2] = __float_as_uint(x2); r0[4 * u + 3] = __float_as_uint(x3);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const uint32_t pk[4] = {gw[e].x, gw[e].y, gw[e].z, gw[e].w};
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                v0[8 * e + 2 * q] = __uint_as_float(r0[8 * e + 2 * q]) * __uint_as_float(pk[q] << 16);
                v0[8 * e + 2 * q + 1] = __uint_as_float(r0[8 * e + 2 * q + 1]) * __uint_as_float(pk[q] & 0xffff0000u);
              }
            }
            if (h16 && row_ok) note_f16_saturation(v0, p.status);
            stage_bf16x32(buf_h, lane, (c & 1) * 4, v0, h16);
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&p.tm_out, bx, col0, row_base);
              if ((c & 1) || c + 1 == n_chunks) tma_store_2d(&p.tm_norm_h, buf_h, n * p.bn + (c >> 1) * 64, row_base);
              bulk_commit();
            }
          }
          if (!okx) break;
          finish_row_norm(p, row, row_ok, m * 4 + quarter, n, n_n_tiles, ss, lane);
          if (lane == 0) bulk_wait_read<0>();         // the staging blocks go back to the alternating use below
          __syncwarp();
          epi_sel = 0;
        } else if (p.norm_gain != nullptr && un.last) {
          // The same fold in the single-block kernel (reached by a folded step only at sm_budget 1): y is read with
          // plain loads; the arithmetic, and so every bit of x, h and the sums, is that of the pair form.
          const float* yrow = p.y_in + size_t(row_ok ? row : 0) * p.N;
          const bool h16 = p.norm_h_f16 != 0;
          float ss = 0.f;
          uint8_t* buf_x = epi_buf;                       // fp32 block of this chunk
          uint8_t* buf_h = epi_buf + EPI_BUF_BYTES;       // 16-bit block of a pair of chunks
          for (int c = 0; c < p.bn / 32; ++c) {
            const int col0 = n * p.bn + c * 32;
            if (col0 >= p.N) break;
            tmem_ld32(taddr + c * 32, r0);
            const int nv = p.N - col0 >= 32 ? 8 : (p.N - col0) >> 2;        // float4s of the chunk inside the row
            float4 yv[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
              yv[e] = row_ok && e < nv ? __ldcg(reinterpret_cast<const float4*>(yrow + col0) + e) : make_float4(0.f, 0.f, 0.f, 0.f);
            uint4 gw[4];                                   // 32 gains (bf16), the same for every row
#pragma unroll
            for (int e = 0; e < 4; ++e)
              gw[e] = 2 * e < nv ? __ldg(reinterpret_cast<const uint4*>(p.norm_gain + col0) + e) : make_uint4(0, 0, 0, 0);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float x0 = __uint_as_float(r0[4 * e]) + yv[e].x, x1 = __uint_as_float(r0[4 * e + 1]) + yv[e].y;
              const float x2 = __uint_as_float(r0[4 * e + 2]) + yv[e].z, x3 = __uint_as_float(r0[4 * e + 3]) + yv[e].w;
              if (e < nv) ss += (x0 * x0 + x1 * x1) + (x2 * x2 + x3 * x3);
              r0[4 * e] = __float_as_uint(x0); r0[4 * e + 1] = __float_as_uint(x1);
              r0[4 * e + 2] = __float_as_uint(x2); r0[4 * e + 3] = __float_as_uint(x3);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const uint32_t pk[4] = {gw[e].x, gw[e].y, gw[e].z, gw[e].w};
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                v0[8 * e + 2 * q] = __uint_as_float(r0[8 * e + 2 * q]) * __uint_as_float(pk[q] << 16);
                v0[8 * e + 2 * q + 1] = __uint_as_float(r0[8 * e + 2 * q + 1]) * __uint_as_float(pk[q] & 0xffff0000u);
              }
            }
            if (h16 && row_ok) note_f16_saturation(v0, p.status);
            if (lane == 0) bulk_wait_read<0>();       // both staging blocks have been read by their last stores
            __syncwarp();
            stage_f32x32(buf_x, lane, r0);
            stage_bf16x32(buf_h, lane, (c & 1) * 4, v0, h16);
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&p.tm_out, buf_x, col0, row_base);
              if ((c & 1) || col0 + 32 >= p.N) tma_store_2d(&p.tm_norm_h, buf_h, n * p.bn + (c >> 1) * 64, row_base);
              bulk_commit();
            }
          }
          finish_row_norm(p, row, row_ok, m * 4 + quarter, n, n_n_tiles, ss, lane);
          if (lane == 0) bulk_wait_read<0>();         // the staging blocks go back to the alternating use below
          __syncwarp();
          epi_sel = 0;
        } else
        for (int c = 0; c < p.bn / 32; ++c) {
          const int col0 = n * p.bn + c * 32;
          if (col0 >= p.N) break;
          tmem_ld32(taddr + c * 32, r0);
          float4 gv[8];
          const int nv = p.N - col0 >= 32 ? 8 : (p.N - col0) >> 2;          // float4s of the chunk inside the row
          if (gate) {                              // requested while the accumulator chunk is on its way
#pragma unroll
            for (int e = 0; e < 8; ++e) gv[e] = e < nv ? __ldg(reinterpret_cast<const float4*>(gate + col0) + e) : make_float4(1.f, 1.f, 1.f, 1.f);
          }
          tmem_ld_wait();
          if (gate) {
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              r0[4 * e] = __float_as_uint(__uint_as_float(r0[4 * e]) * gv[e].x);
              r0[4 * e + 1] = __float_as_uint(__uint_as_float(r0[4 * e + 1]) * gv[e].y);
              r0[4 * e + 2] = __float_as_uint(__uint_as_float(r0[4 * e + 2]) * gv[e].z);
              r0[4 * e + 3] = __float_as_uint(__uint_as_float(r0[4 * e + 3]) * gv[e].w);
            }
          }
          if (lane == 0) bulk_wait_read<1>();     // the block staged two chunks ago has been read
          __syncwarp();
          uint8_t* buf = epi_buf + epi_sel * EPI_BUF_BYTES;
          stage_f32x32(buf, lane, r0);
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            if (add) tma_reduce_add_2d(&p.tm_out, buf, col0, row_base);
            else tma_store_2d(&p.tm_out, buf, col0, row_base);
            bulk_commit();
          }
          epi_sel ^= 1;
        }
        if (ordered && !(ks == 0 && un.last) && lane == 0) {    // a tile with a single segment needs no turn
          bulk_wait<0>();                     // this segment's adds have been performed
          __threadfence();
          st_release(turn, un.last ? 0 : ks + 1);   // the last segment leaves the word at zero
        }
      } else if (p.mode == kGemmGateUp) {
        for (int c = 0; c < 4; ++c) {
          const int col0 = n * 128 + c * 32;
          if (col0 >= p.N) break;
          tmem_ld32(taddr + c * 32, r0);          // gate
          tmem_ld32(taddr + 128 + c * 32, r1);    // up
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float g = __uint_as_float(r0[e]) * rs, u = __uint_as_float(r1[e]) * rs;
            v0[e] = __fdividef(g * u, 1.f + __expf(-g));   // silu(g) * u
          }
          if (p.act_f16) note_f16_saturation(v0, p.status);
          uint8_t* buf = epi_buf + epi_sel * EPI_BUF_BYTES;
          if ((c & 1) == 0) {
            if (lane == 0) bulk_wait_read<1>();
            __syncwarp();
          }
          stage_bf16x32(buf, lane, (c & 1) * 4, v0, p.act_f16 != 0);
          const bool block_done = (c & 1) || col0 + 32 >= p.N;
          if (block_done) {                       // 64 columns staged (or the ragged end of the row)
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
              tma_store_2d(&p.tm_act, buf, n * 128 + (c >> 1) * 64, row_base);
              bulk_commit();
            }
            epi_sel ^= 1;
          }
        }
      } else {
        const int pos = row_ok ? p.tok_pos[row] : 0;
        const int slot = row_ok ? p.tok_slot[row] : 0;
        const int half_dh = Dh >> 1;
        const int qkv_w = gemm_qkv_width(p);
        for (int half = 0; half < qkv_w / 128; ++half) {
          int vcol = n * qkv_w + half * 128;      // virtual column of this half in [q | k | v]
          if (vcol >= p.N) break;
          int region = 0;
          if (vcol >= p.q_dim) { region = 1; vcol -= p.q_dim; }
          if (region == 1 && vcol >= p.kv_dim) { region = 2; vcol -= p.kv_dim; }
          const __nv_bfloat16* bias = p.qkv_bias[region];      // of this region's projection, or null
          if (region == 2) {
            for (int c = 0; c < 4; ++c) {
              tmem_ld32(taddr + half * 128 + c * 32, r0);
              tmem_ld_wait();
              if (p.in_row_rs) scale32(r0, rs);
              if (bias) add_bias32(r0, bias + vcol + c * 32);
              if (row_ok) {
#pragma unroll
                for (int e = 0; e < 32; ++e) v0[e] = __uint_as_float(r0[e]);
                const int col = vcol + c * 32;
                store_bf16x32(cache_ptr(p.v_cache, slot, col / Dh, p.n_kv_heads, Dh, col % Dh), v0, 32);
              }
            }
          } else {
            if (region == 0) {                    // both staging blocks are about to be refilled
              if (lane == 0) bulk_wait_read<0>();
              __syncwarp();
            }
            for (int j = 0; j < 2; ++j) {
              const int lo = Dh == 128 ? j : 2 * j, hi = lo + (Dh == 128 ? 2 : 1);
              const int i0 = Dh == 128 ? 32 * j : 0;       // index of the first rotation pair
              tmem_ld32(taddr + half * 128 + lo * 32, r0);
              tmem_ld32(taddr + half * 128 + hi * 32, r1);
              tmem_ld_wait();
              if (p.in_row_rs) {
                scale32(r0, rs);
                scale32(r1, rs);
              }
              if (bias) {                                        // the bias comes before the rotation
                add_bias32(r0, bias + vcol + lo * 32);
                add_bias32(r1, bias + vcol + hi * 32);
              }
              const float2* cs = p.rope + size_t(pos) * half_dh + i0;
#pragma unroll
              for (int e = 0; e < 32; e += 2) {
                const float4 t = *reinterpret_cast<const float4*>(cs + e);   // cos,sin of pairs e, e+1
                const float a0 = __uint_as_float(r0[e]), b0 = __uint_as_float(r1[e]);
                const float a1 = __uint_as_float(r0[e + 1]), b1 = __uint_as_float(r1[e + 1]);
                v0[e] = a0 * t.x - b0 * t.y;
                v1[e] = b0 * t.x + a0 * t.y;
                v0[e + 1] = a1 * t.z - b1 * t.w;
                v1[e + 1] = b1 * t.z + a1 * t.w;
              }
              if (region == 0) {
                // chunk ch of the half belongs to 64-column block ch / 2, units 4 (ch % 2) ..
                stage_bf16x32(epi_buf + (lo >> 1) * EPI_BUF_BYTES, lane, (lo & 1) * 4, v0);
                stage_bf16x32(epi_buf + (hi >> 1) * EPI_BUF_BYTES, lane, (hi & 1) * 4, v1);
              } else if (row_ok) {
                const int col_lo = vcol + lo * 32, col_hi = vcol + hi * 32;
                store_bf16x32(cache_ptr(p.k_cache, slot, col_lo / Dh, p.n_kv_heads, Dh, col_lo % Dh), v0, 32);
                store_bf16x32(cache_ptr(p.k_cache, slot, col_hi / Dh, p.n_kv_heads, Dh, col_hi % Dh), v1, 32);
              }
            }
            if (region == 0) {
              fence_proxy_async();
              __syncwarp();
              if (lane == 0) {
                tma_store_2d(&p.tm_q, epi_buf, vcol, row_base);
                tma_store_2d(&p.tm_q, epi_buf + EPI_BUF_BYTES, vcol + 64, row_base);
                bulk_commit();
              }
            }
          }
        }
      }
      // this warp has drained its rows of the accumulator: tell the MMA issuer (in the leader block)
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) mbar_arrive_cluster(mapa_u32(smem_u32(&tempty[acc]), 0));
        else mbar_arrive(&tempty[acc]);
      }
      acc ^= 1;
      if (acc == 0) acc_ph ^= 1;
    }
    if (lane == 0) bulk_wait<0>();            // every output block has been written
  }

  // ------------------------------------------------------------- teardown --
  __syncwarp();
  if (*abort_flag) drain_after_abort();
  tc_fence_before_sync();
  __syncthreads();
  if (PAIR) cluster_sync_all();               // neither block leaves while the other may still reach into it
  if (warp == 1) {
    tc_fence_after_sync();
    if (PAIR) tmem_dealloc_pair(tmem_base, TMEM_COLS);
    else tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

__global__ void __launch_bounds__(GEMM_THREADS, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
  gemm_body<false>(p);
}
// Two blocks per cluster, one 256 x 256 tile per pair.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
    gemm_pair_kernel(const __grid_constant__ GemmParams p) {
  gemm_body<true>(p);
}

}  // namespace

cudaError_t gemm_set_attributes() {
  cudaError_t e = set_kernel_smem(gemm_pair_kernel, GEMM_SMEM);
  if (e != cudaSuccess) return e;
  return set_kernel_smem(gemm_kernel, GEMM_SMEM);
}

int gemm_pick_bn(int M, int N, int sm_count) {
  // Time of a launch ~ waves x time of one tile.  A tile's MMA work is proportional to its width, but the
  // operand feed is not (the 128-row A tile is fetched whatever the width, and narrow tiles leave less
  // time to hide the fetch): measured on B200, a 224-wide tile takes 0.95 and a 128-wide tile 0.80 of a
  // 256-wide one, i.e. about 0.6 + 0.4 * bn / 256.  The choice depends on the shape and on the device's
  // SM count only -- never on the SM budget -- so that the same tiles are computed at every budget.
  const int m_tiles = (M + BM - 1) / BM;
  int best = BN;
  double best_cost = 1e30;
  for (int bn = 256; bn >= 128; bn -= 32) {
    const int tiles = m_tiles * ((N + bn - 1) / bn);
    const int waves = (tiles + sm_count - 1) / sm_count;
    const double cost = double(waves) * (0.6 + 0.4 * bn / 256.0);
    if (cost < best_cost - 1e-9) {
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

int gemm_pick_ksplit(int M, int N, int K, int bn, int sm_count) {
  // Few tiles (small M): split K so that more SMs stream a share of the weights.  The splits of a tile add
  // their partial sums in split order, one after the other.  Measured on B200 at 64 rows (bn = 128): a block streams
  // a 64-wide K block in about 0.36 us, a link of the chain costs about 3.5 us -- the time of ten K blocks, which is
  // how much longer each split is than the one before it (gemm_split_begin), so that only the last link is exposed.
  // The split count minimises gemm_ksplit_cost_us over ks = 1 .. 8.  Depends on the shape and the device only, never
  // on the SM budget.
  const int tiles = ((M + BM - 1) / BM) * ((N + bn - 1) / bn);
  const int k_blocks = (K + BK - 1) / BK;
  int best = 1;
  double best_cost = 1e30;
  for (int ks = 1; ks <= 8 && ks <= k_blocks; ++ks) {
    if (gemm_split_begin(k_blocks, ks, ks - 1) >= k_blocks) continue;      // an empty last split
    const int waves = (tiles * ks + sm_count - 1) / sm_count;
    const double cost = gemm_ksplit_cost_us(k_blocks, ks, waves);
    if (cost < best_cost - 1e-9) {
      best_cost = cost;
      best = ks;
    }
  }
  return best;
}

int gemm_pick_stream_k(int M, int N, int K, int sm_count) {
  // Whole 256 x 256 tiles on W pairs take ceil(tiles / W) rounds; cutting the K blocks of all tiles into W equal
  // runs takes tiles / W rounds' worth, at the price of a second (ordered) add for the tiles that a cut falls into.
  // Worth it when the last round would be under about 90 % full and K is long: a run that ends inside a tile costs
  // that tile a second epilogue (the 256 x 256 fp32 block leaves by TMA add-reductions, about a third of the main
  // loop's time at K = 3584), and a short head or tail segment cannot hide its epilogue behind the next main loop.
  // Measured on B200 (per launch, whole tiles -> equal runs): 126 tiles of K = 18944 on 74 pairs (1.70 rounds run
  // as 2) 254 -> 233 us at equal clocks; 184 tiles of K = 5632 (2.49 run as 3) 114 -> 104 us; but 126 tiles of
  // K = 3584 62 -> 64 us and 184 tiles of K = 2048 53 -> 52 us: no gain below about 64 K blocks.
  const int W = sm_count / 2;
  const int tiles = ((M + 2 * BM - 1) / (2 * BM)) * ((N + BN - 1) / BN);
  const int k_blocks = (K + BK - 1) / BK;
  if (W < 1 || tiles * 8 > kGemmTurnWords || k_blocks < 64) return 0;
  if (tiles * 2 < W) return 0;                       // few tiles: single blocks with a K split serve better
  const int rounds = (tiles + W - 1) / W;
  return double(tiles) / W < 0.92 * rounds ? W : 0;
}

cudaError_t launch_gemm(const GemmParams& p, int sm_budget, cudaStream_t stream) {
  const int n_m_tiles = (p.M + BM - 1) / BM;
  const int n_n_tiles = gemm_n_tiles(p);
  const int n_tiles = n_m_tiles * n_n_tiles * (p.mode == kGemmResid && p.ksplit > 1 ? p.ksplit : 1);
  if (n_tiles <= 0) return cudaSuccess;
  if (p.pair && sm_budget >= 2) {
    // pairs of blocks (clusters of two SMs) on 256 x 256 tiles; an odd budget leaves one SM unused
    const int pair_tiles = ((p.M + 2 * BM - 1) / (2 * BM)) * n_n_tiles;
    const int pairs = p.mode == kGemmResid && p.stream_k_slots > 0 ? p.stream_k_slots : pair_tiles;
    const int grid = 2 * (pairs < sm_budget / 2 ? pairs : sm_budget / 2);
    return launch_step_kernel(gemm_pair_kernel, grid, GEMM_THREADS, GEMM_SMEM, stream, p.overlap != 0, p);
  }
  const int grid = n_tiles < sm_budget ? n_tiles : sm_budget;
  return launch_step_kernel(gemm_kernel, grid, GEMM_THREADS, GEMM_SMEM, stream, p.overlap != 0, p);
}

}  // namespace hs
