// Launcher interfaces of the step's kernels.  Every launcher enqueues one persistent kernel of at most
// `sm_budget` thread blocks (one per SM: each block asks for more than half of an SM's shared memory)
// on `stream` and returns the launch status.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace hs {

// Dynamic shared memory every kernel requests at least, so that two blocks (of this or of a co-running
// stage's kernel) never share an SM: more than half of the 227 KB an SM offers.
constexpr int kMinSmemBytes = 117 * 1024;
// Warps per block of the decode attention kernel (each works through one item at a time); the planner sizes its
// work items for sm_count x this many warps.
constexpr int kDecodeKernelWarps = 8;

// ------------------------------------------------------------------ GEMM --
// out = A[M,K] * W^T with W given as up to three row blocks [rows, K] (bf16, K contiguous).  The output
// tile is 128 x 256 "virtual" columns; each 128-column half of a tile is fetched from one weight matrix.
enum GemmMode : int {
  kGemmResid = 0,   // out[M,N] fp32 (+)= A W^T: TMA store, or TMA add-reduction into out (out-proj, down)
  kGemmQkv = 1,     // virtual columns [q | k | v]; RoPE on q,k; q -> bf16 buffer, k,v -> paged cache
  kGemmGateUp = 2   // tile = 128 gate columns + the same 128 up columns; act = silu(gate) * up -> bf16
};

struct GemmParams {
  CUtensorMap tm_a;          // activations [rows >= M, K], box 64 x 128
  CUtensorMap tm_b[3];       // weights, box 64 x 128: Resid {W}, Qkv {Wq, Wk, Wv}, GateUp {Wgate, Wup}
  int M, N, K;               // N: Resid output width; Qkv (Hq + 2 Hkv) * Dh; GateUp F (activation width)
  int mode;
  int ab_f16;                // 1: both operands hold fp16 values; 0: both bf16
  int a_box_rows;            // rows of tm_a's box: 128, or 64 / 32 when M is that small (0 means 128); single blocks only
  int overlap;               // 1: launch so that the set-up overlaps the previous kernel's drain
  int pair;                  // 1: run on pairs of SMs (256 x 256 tiles, bn = 256, no K split) when the budget allows
  // Resid
  CUtensorMap tm_out;        // fp32 [M, N], box 32 x 32, 128-byte swizzle (rows past M are clipped)
  int accumulate;            // 1: out += A W^T (the residual add), 0: out = A W^T
  int bn;                    // tile width of this launch (gemm_pick_bn); 256 when unused
  int ksplit;                // K splits per output tile, added in split order (gemm_pick_ksplit); 0/1 = none
  int stream_k_slots;        // pairs only: > 0 = cut the tiles' K blocks into this many equal runs (gemm_pick_stream_k)
  int* tile_turn;            // [tiles * 4] ([tiles * 8] on pairs) whose-turn words for the ordered adds; zero at entry and at exit
  // Qkv
  int q_dim, kv_dim, head_dim, n_kv_heads;
  CUtensorMap tm_q;          // bf16 q [M, q_dim], box 64 x 32, 128-byte swizzle
  __nv_bfloat16* k_cache;    // this layer's K pages: [page][kv_head][16][Dh]
  __nv_bfloat16* v_cache;
  const int32_t* tok_pos;    // [M]
  const int32_t* tok_slot;   // [M]
  const float2* rope;        // [max_position][Dh/2] (cos, sin)
  const __nv_bfloat16* qkv_bias[3];   // optional biases of the q, k, v projections ([q_dim], [kv_dim], [kv_dim]); null = none
  // Resid, optional: out += gate * (A W^T) with the gate vector of the row's sequence: gate_mod is this layer's
  // fp32 [max_seqs][6][N], gate_which the row of the gate vector (2 or 5), tok_seq the sequence of every row
  const float* gate_mod;
  const int32_t* tok_seq;
  int gate_which;
  // GateUp
  CUtensorMap tm_act;        // bf16 act [M, N], box 64 x 32, 128-byte swizzle
  int* status;               // device status word; with act_f16 the word after it counts saturated act values
  int act_f16;               // GateUp: 1 = write act as fp16, 0 = bf16
  int* smid_log;             // nullable: SM census slots of this launch (see log_smid)
  // RMSNorm folded into the GEMMs around it: rmsnorm(x) W^T = diag(r) ((x o g) W^T), r = rsqrt(mean(x^2) + eps).
  //   Resid, producing side (norm_gain non-null): the tile's final segment does not add-reduce its block into the
  //   output but reads it, adds, writes x back and, from the same registers, emits the next GEMM's A operand
  //   h = 16-bit(x o g) (not yet normalised) and the sum of x^2 over the tile's columns, one partial per (row, tile
  //   column), into row_ss[row * ss_stride + tile column]; the warp that delivers a row group's last tile column sums
  //   the partials in tile-column order and writes r into row_rs[row] (row_group_done: one counter per 32 rows,
  //   zero at entry and at exit).
  const __nv_bfloat16* norm_gain;   // [N] gains of the norm that follows, or null
  CUtensorMap tm_norm_h;     // h [M, N] 16-bit, box 64 x 32, 128-byte swizzle
  float* row_ss;             // [M][ss_stride]
  int ss_stride;
  float* row_rs;             // [M] r of every row, for the consuming GEMM
  int* row_group_done;       // [ceil(M / 32)]
  const float* y_in;         // the output as plain memory (the residual stream to read)
  int norm_h_f16;            // 1 = h in fp16, 0 = bf16
  //   Qkv / GateUp, consuming side (in_row_rs non-null): every accumulator row is scaled by r of its token before
  //   bias / RoPE / SiLU.
  const float* in_row_rs;    // [M]
  float norm_eps;            // producing side: eps of the norm that follows
};
cudaError_t launch_gemm(const GemmParams& p, int sm_budget, cudaStream_t stream);
cudaError_t gemm_set_attributes();
// Tile width for a Resid-mode GEMM of this shape on a device with sm_count SMs (budget independent).
int gemm_pick_bn(int M, int N, int sm_count);
int gemm_pick_ksplit(int M, int N, int K, int bn, int sm_count);
// Where split i (0 .. ks) of a tile's k_blocks begins.  The splits add their sums one after the other, a link of that
// chain costing about as long as kSplitSkew K blocks take to stream; so each split is that much longer than the one
// before it and finishes just when its turn comes, instead of all finishing together and then queueing.  Equal
// lengths when K is too short for that.  A function of the shape only.
constexpr int kSplitSkew = 10;
__host__ __device__ inline int gemm_split_begin(int k_blocks, int ks, int i) {
  if (i >= ks) return k_blocks;
  const int tri = kSplitSkew * ks * (ks - 1) / 2;
  if (ks < 2 || k_blocks < tri + ks * kSplitSkew) {
    const int per = (k_blocks + ks - 1) / ks;
    return i * per < k_blocks ? i * per : k_blocks;
  }
  return i * ((k_blocks - tri) / ks) + kSplitSkew * i * (i - 1) / 2;
}
// Modelled time (us) of a K-split residual GEMM of `waves` rounds on single blocks: the longest split's stream and
// what of the chain of adds is not hidden behind it.
inline double gemm_ksplit_cost_us(int k_blocks, int ks, int waves) {
  const int last = k_blocks - gemm_split_begin(k_blocks, ks, ks - 1);
  const bool skewed = gemm_split_begin(k_blocks, ks, 1) != (k_blocks + ks - 1) / ks || ks == 1;
  return double(waves) * last * 0.36 + (ks > 1 ? (skewed ? 3.5 : (ks - 1) * 3.5) : 0.0);
}
// Runs for the stream-K form of a Resid-mode GEMM on pairs (one per pair of the device), or 0 when whole tiles
// already fill their waves well enough (budget independent).
int gemm_pick_stream_k(int M, int N, int K, int sm_count);
// The same three GEMMs for steps of at most 64 rows (gemm_skinny.cu): weight streaming on plain loads and
// warp-level MMAs, one block per 32 output columns and the whole K range, no K split across blocks.
struct SkinnyParams {
  const void* a;             // activations [rows >= T, K], 16-bit (fp16 or bf16 as ab_f16 says), row-major
  const void* w[3];          // Resid {W}, Qkv {Wq, Wk, Wv}, GateUp {Wgate, Wup}; 16-bit [out, K] row-major
  int T, K, N;               // N: Resid output width; Qkv (Hq + 2 Hkv) * Dh; GateUp F
  int mode, ab_f16, overlap;
  float* y;                  // Resid: fp32 [T, N]
  int accumulate;            // Resid: 1: y += A W^T, 0: y = A W^T
  int q_dim, kv_dim, head_dim, n_kv_heads;      // Qkv
  __nv_bfloat16* q_out;      // bf16 [T, q_dim]
  __nv_bfloat16* k_cache;
  __nv_bfloat16* v_cache;
  const int32_t* tok_pos;
  const int32_t* tok_slot;
  const float2* rope;
  const __nv_bfloat16* qkv_bias[3];   // optional, as in GemmParams
  const float* gate_mod;     // Resid, optional, as in GemmParams
  const int32_t* tok_seq;
  int gate_which;
  __nv_bfloat16* act;        // GateUp: 16-bit [T, N]
  int act_f16;
  int* status;               // nullable: the stage's device status words (the second one counts fp16 saturations)
  int* smid_log;
  // RMSNorm folded into the GEMMs around it, as in GemmParams (rmsnorm(x) W^T = diag(r) ((x o g) W^T)).
  //   Resid, producing side (norm_gain non-null): the epilogue also emits h = 16-bit(y o g) for the next GEMM and the
  //   sum of y^2 over the unit's 32 columns into row_ss[row * ss_stride + unit].  When the GEMM behind the norm is the
  //   tiled kernel (units_done non-null), the block that delivers the last unit (units_done: one counter, zero at entry
  //   and at exit) sums every row's partials and writes r = rsqrt(mean(y^2) + norm_eps) into row_rs[row]; when it is
  //   this kernel, that GEMM sums the partials itself (in_row_ss) and the producer's tail stays short.
  const __nv_bfloat16* norm_gain;   // [N]
  __nv_bfloat16* norm_h;     // 16-bit [T, N]
  int norm_h_f16;
  float* row_ss;             // [T][ss_stride], ss_stride >= N / 32
  int ss_stride;
  float* row_rs;             // [T]
  int* units_done;
  float norm_eps;            // both sides
  //   Qkv / GateUp, consuming side: every output row is scaled by r of its token before bias / RoPE / SiLU; r comes
  //   from in_row_rs[row], or (in_row_ss non-null) from the K / 32 partials in_row_ss[row * (K / 32) + i], which four
  //   threads per row add in the order the producer's last block would have.
  const float* in_row_rs;    // [T]
  const float* in_row_ss;    // [T][K / 32]
};
// True when the skinny kernel covers this shape (few rows, K a multiple of 32, widths it can tile).
bool gemm_skinny_supports(int T, int K, int N, int mode, int head_dim);
// True when it is also expected to be faster than the tiled kernel for this shape (budget independent).
bool gemm_skinny_wins(int T, int K, int N, int mode, int head_dim, int sm_count);
cudaError_t launch_gemm_skinny(const SkinnyParams& p, int sm_budget, cudaStream_t stream);
cudaError_t gemm_skinny_set_attributes();
constexpr int kGemmTurnWords = 4096;   // capacity of the whose-turn array: splits are used only when tiles * 4 fits

// ---------------------------------------------------------------- RMSNorm --
// h[t,:] = bf16(x[t,:] * rsqrt(mean(x[t,:]^2) + eps) * g).  x comes either as bf16 (x_bf16, first layer;
// x_f32_out then receives the widened copy that starts the fp32 residual stream) or as fp32 (x_f32).
struct NormParams {
  const __nv_bfloat16* x_bf16;
  const float* x_f32;
  float* x_f32_out;
  const __nv_bfloat16* gain;
  __nv_bfloat16* h;
  int T, d;
  float eps;
  const int* row_index;      // nullable: input row of output row t is row_index[t] (device int32 [T]); else t
  // optional modulation of a conditioned block: h = rmsnorm(x) g (1 + scale) + shift with the vectors of the
  // row's sequence; mod is this layer's fp32 [max_seqs][6][d], mod_which the row of the shift vector (0 or 3,
  // the scale follows it), tok_seq the sequence of every row.  mod null = none.
  const float* mod;
  const int32_t* tok_seq;
  int mod_which;
  int h_f16;                 // 1 = write h as fp16, 0 = bf16
  int overlap;               // 1: launch so that the set-up overlaps the previous kernel's drain
  int* status;               // device status word (bounded waits report HS_ERR_TIMEOUT here)
  int* smid_log;             // nullable: SM census slots of this launch
};
cudaError_t launch_rmsnorm(const NormParams& p, int sm_budget, cudaStream_t stream);

// Embedding lookup and greedy sampling (head.cu).
struct EmbedParams {
  const int32_t* tokens;           // device [n]
  const __nv_bfloat16* table;      // [vocab, d]
  __nv_bfloat16* x_out;            // [n, d]
  int n, vocab, d;
  int* status;                     // receives HS_ERR_INVALID_ARG for an id outside the table
};
struct ArgmaxParams {
  const float* logits;             // [n, vocab]
  int32_t* tokens;                 // [n]: lowest index of each row's maximum
  int n, vocab;
};
cudaError_t head_set_attributes();
cudaError_t launch_embed(const EmbedParams& p, int sm_budget, cudaStream_t stream);
cudaError_t launch_argmax(const ArgmaxParams& p, int sm_budget, cudaStream_t stream);
// dst[i] = fp16(src[i]) for n bf16 values (n a multiple of 8, both 16-byte aligned); used once per weight
// matrix when a stage is created
cudaError_t launch_bf16_to_f16(const void* src, void* dst, size_t n, cudaStream_t stream);
cudaError_t norm_set_attributes();

// -------------------------------------------------------------- attention --
struct AttnParams {
  CUtensorMap tm_kv;               // whole pool as rows of Dh bf16: box 64 x 16, 128-byte swizzle
  CUtensorMap tm_q;                // q [max_tokens, q_dim]: box 64 x prefill_tokens, 128-byte swizzle
  int prefill_tokens;              // tokens per prefill work item
  int o_f16;                       // 1 = write o as fp16, 0 = bf16 (q, K, V are always bf16)
  int overlap;               // 1: launch so that the set-up overlaps the previous kernel's drain
  const __nv_bfloat16* q;          // [T, q_dim] (after RoPE)
  __nv_bfloat16* o;                // [T, q_dim]
  int n_q_heads, n_kv_heads, head_dim, num_pages, max_pages_per_seq, layer;
  const int32_t* seq_tok0;
  const int32_t* seq_ctx;
  const int32_t* seq_qlen;   // new tokens per sequence (prefill kernel, bidirectional only)
  int bidirectional;         // prefill kernel: 1 = no causal mask, a row sees every key of its sequence
  const int32_t* block_tables;
  const int32_t* prefill_items;    // two int4 per item: {seq, kv head, first token, tokens} {cached tokens, first token
                                   //                    row and new tokens of the sequence, 0}
  int n_prefill_items;
  const int32_t* decode_items;     // two int4 per item: {decode row, kv head, first key, end key}
                                   //                    {seq, token row, first item of its group, splits}
  int n_decode_items;
  int decode_group;                // 1: the items are eight page slices per (sequence, KV head) group, group-major; a block
                                   //    works whole groups and merges their slices in shared memory (small batches)
  const int32_t* decode_rows;      // int4 per decode sequence
  int n_decode_rows;
  float* part_o;                   // [max_decode_items][16][Dh] unnormalised partial outputs
  float* part_ml;                  // [max_decode_items][16][2]  running max (log2 domain) and sum
  int* counters;                   // two work-queue heads of this layer (prefill, decode), zero at entry
  int* group_done;                 // [n_decode_rows * n_kv_heads] finished splits per group, zero at entry
                                   // and left at zero by the kernel
  int* status;
  int* smid_log;                   // nullable: SM census slots; prefill uses [0, 160), decode [160, 320)
};
// ------------------------------------------------- one-launch small step --
// A whole step of at most 16 decode rows whose four projections run on the weight-streaming kernel, as ONE
// cooperative launch of at most sm_budget blocks: per layer QKV -> decode attention -> out-projection -> gate/up ->
// down-projection, the phases separated by bounded grid-wide barriers (a counter in device memory), each phase the
// same device function with the same unit / item decomposition as the kernel of its own, so that the results are
// the same bits.  The RMSNorms are folded into the projections (SkinnyParams); the first norm of the step is
// launched in front of it.
struct SmallLayer {                // one layer's constants, in device memory (written with the step's metadata)
  const void* w_q; const void* w_k; const void* w_v; const void* w_o;     // 16-bit operand copies, [out, in]
  const void* w_gate; const void* w_up; const void* w_down;
  const __nv_bfloat16* g_attn; const __nv_bfloat16* g_mlp;
  const __nv_bfloat16* bias[3];    // optional q, k, v biases
};
struct SmallStepParams {
  AttnParams attn;                 // the decode attention's arguments (layer and counters are set per layer)
  const SmallLayer* layers;
  int n_layers, T, d, F, f16;
  int q_dim, kv_dim, head_dim, n_kv_heads;
  float* x;                        // fp32 residual stream [T, d] (the caller's y_out)
  __nv_bfloat16* h; __nv_bfloat16* q; __nv_bfloat16* o; __nv_bfloat16* act;
  __nv_bfloat16* kv_pool; size_t layer_kv_elems;
  const int32_t* tok_pos; const int32_t* tok_slot; const float2* rope;
  int* counters;                   // [n_layers * 2] queue heads, zero at entry
  float* row_ss; float eps;        // partial sums of squares of the folded norms [T][d / 32]; eps of the norms
  int* grid_bar;                   // one word, zero at entry: blocks arrived at the grid barriers so far
  int* status; int* smid_log;
};
cudaError_t launch_small_step(const SmallStepParams& p, int sm_budget, cudaStream_t stream);
cudaError_t small_step_set_attributes();

cudaError_t launch_attention_prefill(const AttnParams& p, int sm_budget, cudaStream_t stream);
cudaError_t launch_attention_decode(const AttnParams& p, int sm_budget, cudaStream_t stream);
cudaError_t attention_set_attributes();
cudaError_t attention_prefill_set_attributes();

}  // namespace hs
