// C ABI of the library: stage object, page allocator front end, step orchestration.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <memory>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "../../include/horizonserve_head.h"
#include "../../include/horizonserve_ops.h"
#include "hs_internal.h"
#include "kernels.h"
#include "ptx.cuh"

namespace hs {
namespace {

constexpr int kRing = 4;   // pinned staging slots for step metadata
constexpr int kRowSsStride = 64;   // partial sums of x^2 kept per token: one per 128-column tile of d_model at most

struct WsLayout {
  size_t rope, h, q, o, act, meta, part_o, part_ml, status, turn, smid, row_ss, row_rs, row_done, w16, w16_layer, total;
};

// elements of the i-th weight matrix of a layer, in the order w_q, w_k, w_v, w_o, w_gate, w_up, w_down
size_t weight_elems(const hs_stage_config_t& c, int i) {
  const size_t d = c.d_model, F = c.d_ffn, q_dim = size_t(c.n_q_heads) * c.head_dim,
               kv_dim = size_t(c.n_kv_heads) * c.head_dim;
  const size_t n[7] = {q_dim * d, kv_dim * d, kv_dim * d, d * q_dim, F * d, F * d, d * F};
  return n[i];
}

WsLayout make_ws_layout(const hs_stage_config_t& c, const MetaLayout& ml) {
  WsLayout w{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    size_t o = off;
    off += align_up(bytes, 1024);
    return o;
  };
  const size_t T = c.max_tokens, q_dim = size_t(c.n_q_heads) * c.head_dim;
  w.rope = take(size_t(c.max_position) * (c.head_dim / 2) * sizeof(float2));
  w.h = take(T * c.d_model * 2);
  w.q = take(T * q_dim * 2);
  w.o = take(T * q_dim * 2);
  w.act = take(T * c.d_ffn * 2);
  w.meta = take(size_t(ml.total) * 4);
  w.part_o = take(size_t(ml.max_decode_items) * 16 * c.head_dim * 4);
  w.part_ml = take(size_t(ml.max_decode_items) * 16 * 2 * 4);
  w.status = take(256);
  w.turn = take(kGemmTurnWords * 4);
  w.smid = take(size_t(HS_PROFILE_CLASSES) * kSmidSlots * 4);
  // partial sums of x^2 per (token, tile column) of a folded RMSNorm; steps of at most 64 rows keep one per 32 columns
  w.row_ss = take(std::max(T * kRowSsStride, size_t(64) * size_t(c.d_model / 32 + 1)) * 4);
  w.row_rs = take(T * 4);                            // r of every token
  w.row_done = take((T / 32 + 2) * 4);               // tile columns delivered per group of 32 token rows
  // fp16 copies of the seven weight matrices of every layer (absent with HS_FLAG_BF16_ACTIVATIONS);
  // within a layer: w_q, w_k, w_v, w_o, w_gate, w_up, w_down, each 1024-byte aligned
  w.w16 = off;
  w.w16_layer = 0;
  if (!(c.flags & HS_FLAG_BF16_ACTIVATIONS)) {
    for (int i = 0; i < 7; ++i) w.w16_layer += align_up(weight_elems(c, i) * 2, 1024);
    take(w.w16_layer * size_t(c.n_layers));
  }
  w.total = off;
  return w;
}

// cuTensorMapEncodeTiled, fetched through the runtime so that the library has no link-time dependency
// on the driver library (it must load on machines without a GPU).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// Row-major matrix [rows, cols] (cols contiguous) of bf16 or fp32; box = 128 bytes of columns x box_rows
// rows, 128-byte swizzle; out-of-range elements read as zero and are clipped on stores.
bool encode_2d(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows, bool f32 = false) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return false;
  const uint64_t esz = f32 ? 4 : 2;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * esz};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / esz), box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
            dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct LayerMaps {
  CUtensorMap wq, wk, wv, wo, wgate, wup, wdown;
};

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    if (prev == dev) prev = -1;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

thread_local std::string g_last_error;
// Records where a CUDA call failed; returns HS_ERR_CUDA so that it can be used in a return statement.
hs_status_t cuda_fail(const char* where, cudaError_t e) {
  g_last_error = std::string(where) + ": " + cudaGetErrorName(e) + " (" + cudaGetErrorString(e) + ")";
  return HS_ERR_CUDA;
}

// Records a failure that has no CUDA error code behind it; returns HS_ERR_CUDA.
hs_status_t fail(const char* what) {
  g_last_error = what;
  return HS_ERR_CUDA;
}

// K splits for a residual GEMM, or 1 when the whose-turn array could not hold its tiles.
int pick_ksplit(int M, int N, int K, int bn, int sm_count) {
  const int tiles = ceil_div(M, 128) * ceil_div(N, bn);
  if (tiles * 4 > kGemmTurnWords) return 1;
  return gemm_pick_ksplit(M, N, K, bn, sm_count);
}

// SM count and compute-capability major of a device, through the attribute queries (cudaGetDeviceProperties
// takes milliseconds, too slow for a per-call check).
bool device_info(int dev, int* sm_count, int* major) {
  return cudaDeviceGetAttribute(sm_count, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
         cudaDeviceGetAttribute(major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess;
}

// Stages may be created and ops called from several host threads (the co-run harness drives each stage from its
// own thread): the table and the attribute calls behind it are serialised.
std::mutex g_attrs_mutex;
bool g_attrs_set[64] = {};
hs_status_t ensure_attributes(int device) {
  std::lock_guard<std::mutex> lock(g_attrs_mutex);
  if (device >= 0 && device < 64 && g_attrs_set[device]) return HS_OK;
  cudaError_t e;
  if ((e = gemm_set_attributes()) != cudaSuccess) return cuda_fail("gemm attributes", e);
  if ((e = norm_set_attributes()) != cudaSuccess) return cuda_fail("rmsnorm attributes", e);
  if ((e = attention_set_attributes()) != cudaSuccess) return cuda_fail("attention attributes", e);
  if ((e = head_set_attributes()) != cudaSuccess) return cuda_fail("head attributes", e);
  if ((e = gemm_skinny_set_attributes()) != cudaSuccess) return cuda_fail("small-step gemm attributes", e);
  if ((e = small_step_set_attributes()) != cudaSuccess) return cuda_fail("one-launch small step attributes", e);
  if (device >= 0 && device < 64) g_attrs_set[device] = true;
  return HS_OK;
}

}  // namespace
}  // namespace hs

using namespace hs;
static_assert(kDecodeWarps == kDecodeKernelWarps, "the planner sizes decode items for the kernel's warp count");

struct hs_stage {
  hs_stage_config_t cfg;
  MetaLayout ml;
  WsLayout ws;
  std::unique_ptr<PageAllocator> alloc;
  std::vector<int32_t> page_stamp;
  int32_t stamp = 0;
  int sm_count = 0;
  uint8_t* ws_dev = nullptr;
  __nv_bfloat16* kv_pool = nullptr;
  std::vector<hs_layer_weights_t> layers;
  struct QkvBias { const __nv_bfloat16* b[3] = {nullptr, nullptr, nullptr}; };
  std::vector<QkvBias> qkv_bias;              // per layer, optional (hs_stage_set_qkv_bias)
  const float* modulation = nullptr;          // optional [n_layers][max_seqs][6][d_model] (hs_stage_set_modulation)
  std::vector<hs_layer_weights_t> operands;   // what the projections read: the fp16 copies, or `layers` itself
  std::vector<LayerMaps> maps;
  CUtensorMap tm_h, tm_o, tm_act, tm_kv;   // operand loads
  CUtensorMap tm_h_s[2], tm_o_s[2], tm_act_s[2];   // the same A operands with 64- and 32-row boxes (small steps)
  CUtensorMap tm_q_st, tm_act_st, tm_h_st; // epilogue stores (box 64 x 32)
  CUtensorMap tm_q_attn;                   // Q tiles of the prefill attention (box 64 x tokens per item)
  int32_t* pinned[kRing] = {};
  cudaEvent_t ev[kRing] = {};
  // The two attention kernels of a layer are independent of each other; with both kinds of work in a step they run
  // side by side, the decode kernel on a stream of the stage's own, forked from and joined to the caller's stream
  cudaStream_t aux_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  bool ev_pending[kRing] = {};
  int ring_pos = 0;
  // optional per-kernel timing
  bool census = false;      // record SM placement of the last step's launches
  bool profile = false;
  struct Timed { int cls; cudaEvent_t a, b; };
  std::vector<Timed> timed;
  std::vector<cudaEvent_t> event_pool;
};

namespace {
// Brackets one launch with events when the stage is being profiled.
struct LaunchTimer {
  hs_stage* s;
  cudaStream_t stream;
  cudaEvent_t a = nullptr, b = nullptr;
  int cls;
  LaunchTimer(hs_stage* st, int c, cudaStream_t str) : s(st), stream(str), cls(c) {
    if (!s->profile) return;
    auto get = [&]() {
      cudaEvent_t e = nullptr;
      if (!s->event_pool.empty()) { e = s->event_pool.back(); s->event_pool.pop_back(); }
      else cudaEventCreate(&e);
      return e;
    };
    a = get(); b = get();
    cudaEventRecord(a, stream);
  }
  ~LaunchTimer() {
    if (!a) return;
    cudaEventRecord(b, stream);
    s->timed.push_back({cls, a, b});
  }
};
}  // namespace

extern "C" {

const char* hs_last_error(void) { return g_last_error.c_str(); }

const char* hs_status_str(hs_status_t s) {
  switch (s) {
    case HS_OK: return "HS_OK";
    case HS_ERR_INVALID_ARG: return "HS_ERR_INVALID_ARG";
    case HS_ERR_INVALID_BUDGET: return "HS_ERR_INVALID_BUDGET";
    case HS_ERR_UNSUPPORTED_SHAPE: return "HS_ERR_UNSUPPORTED_SHAPE";
    case HS_ERR_OUT_OF_PAGES: return "HS_ERR_OUT_OF_PAGES";
    case HS_ERR_BAD_BLOCK_TABLE: return "HS_ERR_BAD_BLOCK_TABLE";
    case HS_ERR_CUDA: return "HS_ERR_CUDA";
    case HS_ERR_TIMEOUT: return "HS_ERR_TIMEOUT";
    case HS_ERR_NO_DEVICE: return "HS_ERR_NO_DEVICE";
    case HS_ERR_UNKNOWN_SEQ: return "HS_ERR_UNKNOWN_SEQ";
  }
  return "HS_ERR_?";
}

size_t hs_kv_pool_bytes(const hs_stage_config_t* cfg) {
  if (!cfg || validate_config(*cfg) != HS_OK) return 0;
  return size_t(cfg->n_layers) * 2 * cfg->num_pages * cfg->n_kv_heads * kPage * cfg->head_dim * 2;
}

size_t hs_workspace_bytes(const hs_stage_config_t* cfg) {
  if (!cfg || validate_config(*cfg) != HS_OK) return 0;
  return make_ws_layout(*cfg, make_meta_layout(*cfg)).total;
}

hs_status_t hs_stage_create(const hs_stage_config_t* cfg, const hs_layer_weights_t* layers, void* kv_pool_dev,
                            void* workspace_dev, hs_stage_t** out) {
  if (!cfg || !out) return HS_ERR_INVALID_ARG;
  *out = nullptr;
  hs_status_t st = validate_config(*cfg);
  if (st != HS_OK) return st;
  const bool host_only = cfg->device < 0;
  if (!host_only) {
    if (!layers || !kv_pool_dev || !workspace_dev) return HS_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(kv_pool_dev) & 255) || (reinterpret_cast<uintptr_t>(workspace_dev) & 255))
      return HS_ERR_INVALID_ARG;
    for (int l = 0; l < cfg->n_layers; ++l) {
      const void* ptrs[9] = {layers[l].g_attn, layers[l].w_q,    layers[l].w_k,  layers[l].w_v,   layers[l].w_o,
                             layers[l].g_mlp,  layers[l].w_gate, layers[l].w_up, layers[l].w_down};
      for (const void* ptr : ptrs)
        if (!ptr || (reinterpret_cast<uintptr_t>(ptr) & 15)) return HS_ERR_INVALID_ARG;
    }
  }
  std::unique_ptr<hs_stage> s(new (std::nothrow) hs_stage());
  if (!s) return HS_ERR_INVALID_ARG;
  s->cfg = *cfg;
  s->ml = make_meta_layout(*cfg);
  s->ws = make_ws_layout(*cfg, s->ml);
  s->alloc.reset(new PageAllocator(cfg->num_pages));
  s->page_stamp.assign(cfg->num_pages, 0);
  if (host_only) {
    *out = s.release();
    return HS_OK;
  }

  DeviceGuard guard(cfg->device);
  if (!guard.ok) return fail("hs_stage_create: cannot make the configured device current");
  int sm_count = 0, major = 0;
  if (!device_info(cfg->device, &sm_count, &major)) return fail("hs_stage_create: device attribute query failed");
  if (major != 10)   // the kernels exist for sm_100a only
    return fail("hs_stage_create: the device is not compute capability 10.x; the kernels are built for sm_100a only");
  s->sm_count = sm_count;
  if ((st = ensure_attributes(cfg->device)) != HS_OK) return st;
  s->ws_dev = static_cast<uint8_t*>(workspace_dev);
  s->kv_pool = static_cast<__nv_bfloat16*>(kv_pool_dev);
  s->layers.assign(layers, layers + cfg->n_layers);

  // RoPE table: angle and cos/sin in double, stored as fp32 (cos, sin)
  const int half = cfg->head_dim / 2;
  std::vector<float2> rope(size_t(cfg->max_position) * half);
  for (int i = 0; i < half; ++i) {
    const double theta = pow(double(cfg->rope_base), -2.0 * i / double(cfg->head_dim));
    for (int pos = 0; pos < cfg->max_position; ++pos) {
      const double phi = double(pos) * theta;
      rope[size_t(pos) * half + i] = make_float2(float(cos(phi)), float(sin(phi)));
    }
  }
  if (cudaMemcpy(s->ws_dev + s->ws.rope, rope.data(), rope.size() * sizeof(float2), cudaMemcpyHostToDevice) !=
          cudaSuccess ||
      cudaMemset(s->ws_dev + s->ws.status, 0, 256) != cudaSuccess ||
      cudaMemset(s->ws_dev + s->ws.turn, 0, kGemmTurnWords * 4) != cudaSuccess ||
      cudaMemset(s->ws_dev + s->ws.row_done, 0, (size_t(cfg->max_tokens) / 32 + 2) * 4) != cudaSuccess)
    return cuda_fail("hs_stage_create: workspace initialisation", cudaGetLastError());

  // tensor maps
  const uint64_t T = cfg->max_tokens, d = cfg->d_model, F = cfg->d_ffn;
  const uint64_t q_dim = uint64_t(cfg->n_q_heads) * cfg->head_dim, kv_dim = uint64_t(cfg->n_kv_heads) * cfg->head_dim;
  bool ok = encode_2d(&s->tm_h, s->ws_dev + s->ws.h, T, d, 128) && encode_2d(&s->tm_o, s->ws_dev + s->ws.o, T, q_dim, 128) &&
            encode_2d(&s->tm_act, s->ws_dev + s->ws.act, T, F, 128);
  for (int i = 0; i < 2 && ok; ++i) {
    const uint32_t rows = i == 0 ? 64 : 32;
    ok = encode_2d(&s->tm_h_s[i], s->ws_dev + s->ws.h, T, d, rows) && encode_2d(&s->tm_o_s[i], s->ws_dev + s->ws.o, T, q_dim, rows) &&
         encode_2d(&s->tm_act_s[i], s->ws_dev + s->ws.act, T, F, rows);
  }
  ok = ok && encode_2d(&s->tm_q_st, s->ws_dev + s->ws.q, T, q_dim, 32) &&
       encode_2d(&s->tm_act_st, s->ws_dev + s->ws.act, T, F, 32) && encode_2d(&s->tm_h_st, s->ws_dev + s->ws.h, T, d, 32);
  ok = ok && encode_2d(&s->tm_q_attn, s->ws_dev + s->ws.q, T, q_dim,
                       prefill_tokens_per_item(cfg->n_q_heads / cfg->n_kv_heads));
  const uint64_t pool_rows = uint64_t(cfg->n_layers) * 2 * cfg->num_pages * cfg->n_kv_heads * kPage;
  ok = ok && encode_2d(&s->tm_kv, s->kv_pool, pool_rows, cfg->head_dim, 16);
  s->maps.resize(cfg->n_layers);
  s->operands = s->layers;
  s->qkv_bias.assign(cfg->n_layers, hs_stage::QkvBias());
  for (int l = 0; l < cfg->n_layers && ok; ++l) {
    LayerMaps& m = s->maps[l];
    hs_layer_weights_t w = s->layers[l];
    if (!(cfg->flags & HS_FLAG_BF16_ACTIVATIONS)) {
      // the projections read fp16 copies of the weights, made here once
      const void* src[7] = {w.w_q, w.w_k, w.w_v, w.w_o, w.w_gate, w.w_up, w.w_down};
      const void** dst[7] = {&w.w_q, &w.w_k, &w.w_v, &w.w_o, &w.w_gate, &w.w_up, &w.w_down};
      uint8_t* at = s->ws_dev + s->ws.w16 + s->ws.w16_layer * size_t(l);
      for (int i = 0; i < 7 && ok; ++i) {
        ok = launch_bf16_to_f16(src[i], at, weight_elems(*cfg, i), nullptr) == cudaSuccess;
        *dst[i] = at;
        at += align_up(weight_elems(*cfg, i) * 2, 1024);
      }
      if (!ok) break;
      s->operands[l] = w;
    }
    ok = encode_2d(&m.wq, w.w_q, q_dim, d, 128) && encode_2d(&m.wk, w.w_k, kv_dim, d, 128) &&
         encode_2d(&m.wv, w.w_v, kv_dim, d, 128) && encode_2d(&m.wo, w.w_o, d, q_dim, 128) &&
         encode_2d(&m.wgate, w.w_gate, F, d, 128) && encode_2d(&m.wup, w.w_up, F, d, 128) &&
         encode_2d(&m.wdown, w.w_down, d, F, 128);
  }
  if (!ok)
    return fail("hs_stage_create: fp16 weight copy or tensor-map encoding failed (cuTensorMapEncodeTiled unavailable, or "
                "a matrix whose row pitch is not a multiple of 16 bytes)");

  if (cudaStreamCreateWithFlags(&s->aux_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&s->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&s->ev_join, cudaEventDisableTiming) != cudaSuccess) {
    const cudaError_t e = cudaGetLastError();
    hs_stage_destroy(s.release());
    return cuda_fail("hs_stage_create: auxiliary stream or event creation", e);
  }
  for (int i = 0; i < kRing; ++i) {
    if (cudaHostAlloc(reinterpret_cast<void**>(&s->pinned[i]), size_t(s->ml.total) * 4, cudaHostAllocDefault) !=
            cudaSuccess ||
        cudaEventCreateWithFlags(&s->ev[i], cudaEventDisableTiming) != cudaSuccess) {
      const cudaError_t e = cudaGetLastError();
      hs_stage_destroy(s.release());
      return cuda_fail("hs_stage_create: pinned staging or event creation", e);
    }
  }
  const cudaError_t sync_err = cudaDeviceSynchronize();
  if (sync_err != cudaSuccess) {
    hs_stage_destroy(s.release());
    return cuda_fail("hs_stage_create: device synchronisation", sync_err);
  }
  *out = s.release();
  return HS_OK;
}

hs_status_t hs_stage_destroy(hs_stage_t* s) {
  if (!s) return HS_ERR_INVALID_ARG;
  if (s->cfg.device >= 0) {
    DeviceGuard guard(s->cfg.device);
    for (int i = 0; i < kRing; ++i) {
      if (s->ev[i]) {
        if (s->ev_pending[i]) cudaEventSynchronize(s->ev[i]);
        cudaEventDestroy(s->ev[i]);
      }
      if (s->pinned[i]) cudaFreeHost(s->pinned[i]);
    }
    if (s->aux_stream) { cudaStreamSynchronize(s->aux_stream); cudaStreamDestroy(s->aux_stream); }
    if (s->ev_fork) cudaEventDestroy(s->ev_fork);
    if (s->ev_join) cudaEventDestroy(s->ev_join);
    for (const hs_stage::Timed& t : s->timed) { cudaEventDestroy(t.a); cudaEventDestroy(t.b); }
    for (cudaEvent_t e : s->event_pool) cudaEventDestroy(e);
  }
  delete s;
  return HS_OK;
}

hs_status_t hs_kv_alloc(hs_stage_t* s, int64_t seq_id, int32_t total_tokens, int32_t* table_out, int32_t cap,
                        int32_t* n_pages_out) {
  if (!s || total_tokens < 0 || cap < 0 || (cap > 0 && !table_out)) return HS_ERR_INVALID_ARG;
  if (ceil_div(total_tokens, kPage) > cap) return HS_ERR_INVALID_ARG;
  const std::vector<int32_t>* table = nullptr;
  const hs_status_t st = s->alloc->grow(seq_id, total_tokens, &table);
  if (st != HS_OK) return st;
  if (int(table->size()) > cap) return HS_ERR_INVALID_ARG;   // owned more than asked before: still reported whole
  for (size_t i = 0; i < table->size(); ++i) table_out[i] = (*table)[i];
  if (n_pages_out) *n_pages_out = int32_t(table->size());
  return HS_OK;
}

hs_status_t hs_kv_free(hs_stage_t* s, int64_t seq_id) {
  if (!s) return HS_ERR_INVALID_ARG;
  return s->alloc->release(seq_id);
}

int32_t hs_kv_free_pages(const hs_stage_t* s) { return s ? s->alloc->free_pages() : -1; }

int32_t hs_stage_sm_count(const hs_stage_t* s) { return s ? s->sm_count : 0; }

hs_status_t hs_stage_plan(hs_stage_t* s, const hs_batch_t* b, int32_t* tok_seq, int32_t* tok_pos, int32_t* tok_slot) {
  if (!s || !b) return HS_ERR_INVALID_ARG;
  std::vector<int32_t> meta(s->ml.total);
  StepPlan plan;
  const hs_status_t st = plan_step(s->cfg, s->ml, *b, s->sm_count, s->page_stamp, ++s->stamp, meta.data(), tok_seq, &plan);
  if (st != HS_OK) return st;
  if (tok_pos) memcpy(tok_pos, meta.data() + s->ml.tok_pos, size_t(plan.n_tokens) * 4);
  if (tok_slot) memcpy(tok_slot, meta.data() + s->ml.tok_slot, size_t(plan.n_tokens) * 4);
  return HS_OK;
}

hs_status_t hs_stage_plan_attention(hs_stage_t* s, const hs_batch_t* b, int32_t* decode_items, int32_t decode_cap,
                                    int32_t* n_decode_items, int32_t* decode_group, int32_t* prefill_items,
                                    int32_t prefill_cap, int32_t* n_prefill_items) {
  if (!s || !b || decode_cap < 0 || prefill_cap < 0) return HS_ERR_INVALID_ARG;
  std::vector<int32_t> meta(s->ml.total);
  StepPlan plan;
  const hs_status_t st = plan_step(s->cfg, s->ml, *b, s->sm_count, s->page_stamp, ++s->stamp, meta.data(), nullptr, &plan);
  if (st != HS_OK) return st;
  if (n_decode_items) *n_decode_items = plan.n_decode_items;
  if (decode_group) *decode_group = plan.decode_group;
  if (n_prefill_items) *n_prefill_items = plan.n_prefill_items;
  if (decode_items)
    memcpy(decode_items, meta.data() + s->ml.decode_items, size_t(std::min(decode_cap, plan.n_decode_items)) * 32);
  if (prefill_items)
    memcpy(prefill_items, meta.data() + s->ml.prefill_items, size_t(std::min(prefill_cap, plan.n_prefill_items)) * 32);
  return HS_OK;
}

int32_t hs_op_gemm_split_begin(int32_t k_blocks, int32_t ks, int32_t i) {
  if (k_blocks < 1 || ks < 1 || i < 0 || i > ks) return -1;
  return gemm_split_begin(k_blocks, ks, i);
}

hs_status_t hs_stage_step(hs_stage_t* s, const hs_batch_t* b, int32_t sm_budget, void* cuda_stream) {
  if (!s || !b) return HS_ERR_INVALID_ARG;
  if (s->cfg.device < 0) return HS_ERR_NO_DEVICE;
  if (sm_budget < 1 || sm_budget > s->sm_count) return HS_ERR_INVALID_BUDGET;
  if (!b->x_in || !b->y_out || (reinterpret_cast<uintptr_t>(b->x_in) & 15) || (reinterpret_cast<uintptr_t>(b->y_out) & 15))
    return HS_ERR_INVALID_ARG;
  const hs_stage_config_t& c = s->cfg;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  DeviceGuard guard(c.device);
  if (!guard.ok) return HS_ERR_CUDA;

  // plan into the next pinned slot (waiting for the copy that last used it)
  const int slot = s->ring_pos;
  if (s->ev_pending[slot]) {
    if (cudaEventSynchronize(s->ev[slot]) != cudaSuccess) return HS_ERR_CUDA;
    s->ev_pending[slot] = false;
  }
  StepPlan plan;
  hs_status_t st = plan_step(c, s->ml, *b, s->sm_count, s->page_stamp, ++s->stamp, s->pinned[slot], nullptr, &plan);
  if (st != HS_OK) return st;
  s->ring_pos = (slot + 1) % kRing;

  {  // the layers' constants for the one-launch small step travel with the metadata (biases may change between steps)
    static_assert(sizeof(SmallLayer) == 24 * 4, "MetaLayout::small_layers holds 24 words per layer");
    SmallLayer* sl = reinterpret_cast<SmallLayer*>(s->pinned[slot] + s->ml.small_layers);
    for (int l = 0; l < c.n_layers; ++l) {
      const hs_layer_weights_t& wo = s->operands[l];
      sl[l] = SmallLayer{wo.w_q, wo.w_k, wo.w_v, wo.w_o, wo.w_gate, wo.w_up, wo.w_down,
                         static_cast<const __nv_bfloat16*>(s->layers[l].g_attn),
                         static_cast<const __nv_bfloat16*>(s->layers[l].g_mlp),
                         {s->qkv_bias[l].b[0], s->qkv_bias[l].b[1], s->qkv_bias[l].b[2]}};
    }
  }
  int32_t* meta = reinterpret_cast<int32_t*>(s->ws_dev + s->ws.meta);
  if (cudaMemcpyAsync(meta, s->pinned[slot], size_t(s->ml.total) * 4, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaEventRecord(s->ev[slot], stream) != cudaSuccess)
    return HS_ERR_CUDA;
  s->ev_pending[slot] = true;

  const int T = plan.n_tokens, d = c.d_model, F = c.d_ffn, Dh = c.head_dim;
  const int q_dim = c.n_q_heads * Dh, kv_dim = c.n_kv_heads * Dh;
  // The fp32 residual stream lives in the caller's y_out for the whole step: the first RMSNorm widens
  // x_in into it and every projection back to d_model is added into it by a TMA reduction.
  float* x = static_cast<float*>(b->y_out);
  CUtensorMap tm_y;
  if (!encode_2d(&tm_y, x, T, d, 32, true)) return HS_ERR_CUDA;
  __nv_bfloat16* h = reinterpret_cast<__nv_bfloat16*>(s->ws_dev + s->ws.h);
  __nv_bfloat16* q = reinterpret_cast<__nv_bfloat16*>(s->ws_dev + s->ws.q);
  __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(s->ws_dev + s->ws.o);
  int* status = reinterpret_cast<int*>(s->ws_dev + s->ws.status);
  const size_t layer_kv_elems = size_t(c.num_pages) * c.n_kv_heads * kPage * Dh;
  cudaError_t e = cudaSuccess;
  const char* where = "";
  // More than one 128-row tile of tokens: a GEMM runs on pairs of SMs (256 x 256 tiles), unless such tiles would
  // occupy less than half of the device's pairs AND its 128-row tiles for single blocks fit one wave: then single
  // blocks occupy more SMs (and a residual GEMM may split K).  A choice by shape, never by budget; the two
  // kernels give the same bits.  Measured at config-3 dimensions, one prefill chunk + decodes (ms per step, all
  // pairs -> this rule): 220 rows 7.41 -> 5.60, 440 rows 9.23 -> 8.63; at 650 rows and more (pair tiles on 57 %
  // of the pairs and up) pairs are the faster form again, a pair tile moving two thirds of the operand bytes of
  // two single tiles.
  const bool use_pair = T > 128;
  auto pair_for = [&](int n_cols, int single_bn) {
    if (!use_pair) return false;
    const bool few_pair_tiles = ceil_div(T, 256) * ceil_div(n_cols, 256) < s->sm_count / 4;
    const bool singles_fit = ceil_div(T, 128) * ceil_div(n_cols, single_bn) <= s->sm_count;
    return !(few_pair_tiles && singles_fit);
  };
  const bool pair_qkv = pair_for(q_dim + 2 * kv_dim, 128), pair_gu = pair_for(2 * F, 256);
  const bool pair_d = pair_for(d, gemm_pick_bn(T, d, s->sm_count));
  const int f16 = (c.flags & HS_FLAG_BF16_ACTIVATIONS) ? 0 : 1;   // format of h, o, act
  // With the whole device as its budget a step has no neighbour to take SMs from, so each kernel is launched
  // such that its set-up overlaps the previous kernel's drain.  With a smaller budget the blocks of the next
  // kernel would wait on SMs outside the budget, so the launches stay strictly serial.  (Not while the
  // per-kernel timers run: an event between two kernels serialises them anyway.)
  const int overlap = (sm_budget == s->sm_count && !s->profile) ? 1 : 0;
  // A operands of a small step are fetched with boxes of 64 or 32 rows instead of 128
  const int a_rows = use_pair ? 128 : (T <= 32 ? 32 : T <= 64 ? 64 : 128);
  const int a_sel = a_rows == 64 ? 0 : 1;
  // Steps of at most 64 rows: a projection runs on the weight-streaming kernel (no K split) where that is the
  // faster one for its shape
  auto skinny = [&](int K, int N, int mode) { return gemm_skinny_wins(T, K, N, mode, Dh, s->sm_count); };
  auto skinny_base = [&](const void* a, int K, int N, int mode) {
    SkinnyParams k{};
    k.a = a; k.T = T; k.K = K; k.N = N; k.mode = mode;
    k.ab_f16 = f16; k.overlap = overlap;
    k.status = status;
    return k;
  };
  // RMSNorm folded into the GEMMs around it (rmsnorm(x) W^T = diag(r) ((x o g) W^T)): the residual GEMM in front of a
  // norm emits h = 16-bit(x o g) and the partial sums of x^2 from its epilogue, the GEMM behind it scales its
  // accumulator rows by r.  Used when all four projections of the step run on pairs of SMs and the stage is not
  // conditioned (a shift between norm and product breaks the factoring); the first norm of a step, which has no
  // GEMM in front of it, stays a kernel.  A choice by shape and stage, never by budget.  Measured on B200 the fold
  // costs each residual GEMM about what the RMSNorm launch it replaces cost (config 2 and 3 steps within 1 % either
  // way, at the full budget and at partial ones); what it buys is two launches per layer.
  const int n_ss_tiles = ceil_div(d, pair_d ? 256 : gemm_pick_bn(T, d, s->sm_count));
  const bool fold_norm = !s->modulation && n_ss_tiles <= kRowSsStride && !skinny(d, q_dim + 2 * kv_dim, kGemmQkv) &&
                         !skinny(q_dim, d, kGemmResid) && !skinny(d, F, kGemmGateUp) && !skinny(F, d, kGemmResid) &&
                         pair_d && pair_qkv && pair_gu;
  // Steps of at most 16 rows: a residual projection on the weight-streaming kernel folds the norm behind it the same
  // way (its epilogue emits h and the row sums, the block that delivers the last unit finalises r); the projection
  // behind the norm -- on either kernel -- scales its rows.  A choice by shape, never by budget.  Measured on B200, the
  // 12-layer talker step: the fold costs a residual GEMM 2 us and saves a launch, which is 2 % slower at the full
  // budget (where launch overlap hides most of a launch) and 11-14 % faster at budgets 112 / 74 / 37, the budgets a
  // downstream stage runs at; at 64 rows (config-3 decode tick: +4 us per out-projection) it is -1.4 % / +2 %, so
  // larger steps keep the separate kernel.
  const bool sk_fold = !s->modulation && T <= 16;
  const bool sk_fold_mlp = sk_fold && skinny(q_dim, d, kGemmResid);
  const bool sk_fold_attn = sk_fold && skinny(F, d, kGemmResid);
  // (a weight-streaming GEMM behind the norm adds the rows' partial sums itself; a tiled one reads r, which the
  // producer's last block then has to finalise)
  auto sk_fold_out = [&](SkinnyParams& k, const void* gain, bool consumer_is_skinny) {
    k.norm_gain = static_cast<const __nv_bfloat16*>(gain);
    k.norm_h = h;
    k.norm_h_f16 = f16;
    k.row_ss = reinterpret_cast<float*>(s->ws_dev + s->ws.row_ss);
    k.ss_stride = d / 32;
    if (!consumer_is_skinny) {
      k.row_rs = reinterpret_cast<float*>(s->ws_dev + s->ws.row_rs);
      k.units_done = reinterpret_cast<int*>(s->ws_dev + s->ws.row_done);
    }
    k.norm_eps = c.rms_eps;
  };
  auto sk_fold_in = [&](SkinnyParams& k) {
    k.in_row_ss = reinterpret_cast<const float*>(s->ws_dev + s->ws.row_ss);
    k.norm_eps = c.rms_eps;
  };
  float* row_ss = reinterpret_cast<float*>(s->ws_dev + s->ws.row_ss);
  auto fold_out = [&](GemmParams& gp, const void* gain) {      // producing side
    gp.norm_gain = static_cast<const __nv_bfloat16*>(gain);
    gp.tm_norm_h = s->tm_h_st;
    gp.row_ss = row_ss;
    gp.ss_stride = kRowSsStride;
    gp.row_rs = reinterpret_cast<float*>(s->ws_dev + s->ws.row_rs);
    gp.row_group_done = reinterpret_cast<int*>(s->ws_dev + s->ws.row_done);
    gp.y_in = x;
    gp.norm_h_f16 = f16;
    gp.norm_eps = c.rms_eps;
  };
  auto fold_in = [&](GemmParams& gp) {                         // consuming side
    gp.in_row_rs = reinterpret_cast<const float*>(s->ws_dev + s->ws.row_rs);
  };
  int* census = s->census ? reinterpret_cast<int*>(s->ws_dev + s->ws.smid) : nullptr;
  if (census && cudaMemsetAsync(census, 0, size_t(HS_PROFILE_CLASSES) * kSmidSlots * 4, stream) != cudaSuccess)
    return HS_ERR_CUDA;
  auto slots = [&](int cls) { return census ? census + cls * kSmidSlots : nullptr; };

  // Split of the SM budget between the two attention kernels when a step has both kinds of work (0 = one after the
  // other).  The decode kernel is bound by the K / V bytes it streams, the prefill kernel by its key blocks; with the
  // rates measured on B200 (about 42 GB/s per SM up to 5.5 TB/s; 1.15 us per block of an item; 12 us per launch)
  //   t_decode(b) = 12 + bytes / min(5.5e6, 42e3 b)    t_prefill(b) = 12 + 1.15 max(longest item, blocks / b)   [us]
  // and the split is the one with the smallest larger time, taken only if that beats running them in turn by 8 %.
  // It moves work between SMs, never between results: both kernels give the same bits at any grid size.
  int decode_sms = 0;
  if (plan.n_prefill_items > 0 && plan.n_decode_items > 0 && sm_budget >= 16 && !s->profile) {   // (per-kernel timing keeps them apart)
    auto t_dec = [&](int b) { return 12.0 + double(plan.decode_kv_bytes) / std::min(5.5e6, 42e3 * b); };
    auto t_pre = [&](int b) { return 12.0 + 1.15 * std::max(double(plan.prefill_longest), double(plan.prefill_blocks) / b); };
    double best = 0.92 * (t_dec(sm_budget) + t_pre(sm_budget));
    for (int b = 4; b <= sm_budget - 4; ++b) {
      const double t = std::max(t_dec(b), t_pre(sm_budget - b));
      if (t < best) { best = t; decode_sms = b; }
    }
  }

  auto make_attn = [&](int l) {
    AttnParams a{};
    a.tm_kv = s->tm_kv;
    a.tm_q = s->tm_q_attn;
    a.prefill_tokens = prefill_tokens_per_item(c.n_q_heads / c.n_kv_heads);
    a.o_f16 = f16;
    a.overlap = overlap;
    a.q = q; a.o = o;
    a.n_q_heads = c.n_q_heads; a.n_kv_heads = c.n_kv_heads; a.head_dim = Dh;
    a.num_pages = c.num_pages; a.max_pages_per_seq = c.max_pages_per_seq; a.layer = l;
    a.seq_tok0 = meta + s->ml.seq_tok0;
    a.seq_ctx = meta + s->ml.seq_ctx;
    a.seq_qlen = meta + s->ml.seq_qlen;
    a.bidirectional = (c.flags & HS_FLAG_BIDIRECTIONAL) ? 1 : 0;
    a.block_tables = meta + s->ml.block_tables;
    a.prefill_items = meta + s->ml.prefill_items;
    a.n_prefill_items = plan.n_prefill_items;
    a.decode_items = meta + s->ml.decode_items;
    a.n_decode_items = plan.n_decode_items;
    a.decode_group = plan.decode_group;
    a.decode_rows = meta + s->ml.decode_rows;
    a.n_decode_rows = plan.n_decode_rows;
    a.part_o = reinterpret_cast<float*>(s->ws_dev + s->ws.part_o);
    a.part_ml = reinterpret_cast<float*>(s->ws_dev + s->ws.part_ml);
    a.counters = meta + s->ml.counters + 2 * l;
    a.group_done = meta + s->ml.group_done;
    a.status = status;
    a.smid_log = slots(2);       // prefill in class 2, decode in class 3 (the next slots)
    return a;
  };
  // A decode-only step of at most 16 rows whose projections all run on the weight-streaming kernel with the norms
  // folded, under a partial budget: after the first norm, ONE cooperative launch does all layers (launch_small_step);
  // the same device functions on the same units and items, so the same bits as the launches below (which is why this
  // choice may look at the budget).  At the full budget the separate launches overlap each other's set-up and are the
  // faster form (talker step 0.40 ms against 0.52); below it they run strictly one after the other (0.58 / 0.60 /
  // 0.75 ms at 112 / 74 / 37 SMs against 0.52 / 0.54 / 0.69 in one launch).  Not while the per-kernel timers run.
  const bool one_launch = sk_fold_mlp && sk_fold_attn && skinny(d, q_dim + 2 * kv_dim, kGemmQkv) && skinny(d, F, kGemmGateUp) &&
                          plan.n_prefill_items == 0 && plan.n_decode_items > 0 && !s->profile && sm_budget < s->sm_count;
  for (int l = 0; l < c.n_layers && e == cudaSuccess; ++l) {
    const hs_layer_weights_t& w = s->layers[l];
    const LayerMaps& m = s->maps[l];
    const hs_layer_weights_t& wo = s->operands[l];

    NormParams np{};
    np.x_bf16 = l == 0 ? static_cast<const __nv_bfloat16*>(b->x_in) : nullptr;
    np.x_f32 = x;
    np.x_f32_out = x;
    np.gain = static_cast<const __nv_bfloat16*>(w.g_attn);
    np.h = h;
    np.T = T;
    np.d = d;
    np.eps = c.rms_eps;
    np.h_f16 = f16;
    np.status = status;
    np.overlap = overlap;
    np.smid_log = slots(0);
    const float* mod_l = s->modulation ? s->modulation + size_t(l) * c.max_seqs * 6 * d : nullptr;
    np.mod = mod_l;
    np.tok_seq = meta + s->ml.tok_seq;
    np.mod_which = 0;
    const bool folded_attn_norm = (fold_norm || sk_fold_attn) && l > 0;   // the previous layer's down-projection produced h and the sums
    if (!folded_attn_norm) { LaunchTimer t(s, 0, stream); where = "rmsnorm"; e = launch_rmsnorm(np, sm_budget, stream); }
    if (e != cudaSuccess) break;
    if (one_launch) {
      SmallStepParams sp{};
      sp.attn = make_attn(0);
      sp.attn.smid_log = nullptr;
      sp.layers = reinterpret_cast<const SmallLayer*>(meta + s->ml.small_layers);
      sp.n_layers = c.n_layers; sp.T = T; sp.d = d; sp.F = F; sp.f16 = f16;
      sp.q_dim = q_dim; sp.kv_dim = kv_dim; sp.head_dim = Dh; sp.n_kv_heads = c.n_kv_heads;
      sp.x = x; sp.h = h; sp.q = q; sp.o = o;
      sp.act = reinterpret_cast<__nv_bfloat16*>(s->ws_dev + s->ws.act);
      sp.kv_pool = s->kv_pool; sp.layer_kv_elems = layer_kv_elems;
      sp.tok_pos = meta + s->ml.tok_pos; sp.tok_slot = meta + s->ml.tok_slot;
      sp.rope = reinterpret_cast<const float2*>(s->ws_dev + s->ws.rope);
      sp.counters = meta + s->ml.counters;
      sp.row_ss = reinterpret_cast<float*>(s->ws_dev + s->ws.row_ss);
      sp.eps = c.rms_eps;
      sp.grid_bar = meta + s->ml.grid_bar;
      sp.status = status;
      sp.smid_log = slots(1);
      where = "small step"; e = launch_small_step(sp, sm_budget, stream);
      // a device or context that cannot hold the grid resident at once (or knows no cooperative launch) takes the
      // separate launches below: the same results
      if (e != cudaErrorCooperativeLaunchTooLarge && e != cudaErrorNotSupported) break;
      cudaGetLastError();
      e = cudaSuccess;
    }

    GemmParams g{};
    g.tm_a = a_rows == 128 ? s->tm_h : s->tm_h_s[a_sel];
    g.a_box_rows = a_rows;
    g.tm_b[0] = m.wq; g.tm_b[1] = m.wk; g.tm_b[2] = m.wv;
    g.M = T; g.N = q_dim + 2 * kv_dim; g.K = d;
    g.mode = kGemmQkv;
    g.ab_f16 = f16;
    g.overlap = overlap;
    g.pair = pair_qkv;
    g.bn = pair_qkv ? 256 : 128;     // small steps: 128-column tiles, twice as many SMs stream the weights
    g.q_dim = q_dim; g.kv_dim = kv_dim; g.head_dim = Dh; g.n_kv_heads = c.n_kv_heads;
    g.tm_q = s->tm_q_st;
    g.k_cache = s->kv_pool + (size_t(l) * 2 + 0) * layer_kv_elems;
    g.v_cache = s->kv_pool + (size_t(l) * 2 + 1) * layer_kv_elems;
    g.tok_pos = meta + s->ml.tok_pos;
    g.tok_slot = meta + s->ml.tok_slot;
    g.rope = reinterpret_cast<const float2*>(s->ws_dev + s->ws.rope);
    for (int i = 0; i < 3; ++i) g.qkv_bias[i] = s->qkv_bias[l].b[i];
    g.status = status;
    g.smid_log = slots(1);
    if (folded_attn_norm) fold_in(g);
    if (skinny(d, q_dim + 2 * kv_dim, kGemmQkv)) {
      SkinnyParams k = skinny_base(h, d, q_dim + 2 * kv_dim, kGemmQkv);
      k.w[0] = wo.w_q; k.w[1] = wo.w_k; k.w[2] = wo.w_v;
      k.q_dim = q_dim; k.kv_dim = kv_dim; k.head_dim = Dh; k.n_kv_heads = c.n_kv_heads;
      k.q_out = q; k.k_cache = g.k_cache; k.v_cache = g.v_cache;
      k.tok_pos = g.tok_pos; k.tok_slot = g.tok_slot; k.rope = g.rope;
      for (int i = 0; i < 3; ++i) k.qkv_bias[i] = g.qkv_bias[i];
      k.smid_log = slots(1);
      if (sk_fold_attn && l > 0) sk_fold_in(k);
      else k.in_row_rs = g.in_row_rs;
      LaunchTimer t(s, 1, stream); where = "qkv gemm"; e = launch_gemm_skinny(k, sm_budget, stream);
    } else { LaunchTimer t(s, 1, stream); where = "qkv gemm"; e = launch_gemm(g, sm_budget, stream); }
    if (e != cudaSuccess) break;

    AttnParams a = make_attn(l);
    if (decode_sms > 0) {
      // side by side: the decode kernel on the stage's own stream with decode_sms of the budget, the prefill kernel on
      // the caller's stream with the rest; both are joined before the out-projection
      AttnParams ad = a;
      ad.overlap = 0;
      if (cudaEventRecord(s->ev_fork, stream) != cudaSuccess || cudaStreamWaitEvent(s->aux_stream, s->ev_fork, 0) != cudaSuccess) {
        e = cudaGetLastError(); where = "attention fork"; break;
      }
      { LaunchTimer t(s, 3, s->aux_stream); where = "decode attention"; e = launch_attention_decode(ad, decode_sms, s->aux_stream); }
      if (e != cudaSuccess) break;
      if (cudaEventRecord(s->ev_join, s->aux_stream) != cudaSuccess) { e = cudaGetLastError(); where = "attention join"; break; }
      { LaunchTimer t(s, 2, stream); where = "prefill attention"; e = launch_attention_prefill(a, sm_budget - decode_sms, stream); }
      if (e != cudaSuccess) break;
      if (cudaStreamWaitEvent(stream, s->ev_join, 0) != cudaSuccess) { e = cudaGetLastError(); where = "attention join"; break; }
    } else {
      if (a.n_prefill_items > 0) { LaunchTimer t(s, 2, stream); where = "prefill attention"; e = launch_attention_prefill(a, sm_budget, stream); }
      if (e != cudaSuccess) break;
      if (a.n_decode_items > 0) { LaunchTimer t(s, 3, stream); where = "decode attention"; e = launch_attention_decode(a, sm_budget, stream); }
      if (e != cudaSuccess) break;
    }

    GemmParams go{};
    go.tm_a = a_rows == 128 ? s->tm_o : s->tm_o_s[a_sel];
    go.a_box_rows = a_rows;
    go.tm_b[0] = m.wo; go.tm_b[1] = m.wo; go.tm_b[2] = m.wo;
    go.M = T; go.N = d; go.K = q_dim;
    go.mode = kGemmResid;
    go.ab_f16 = f16;
    go.overlap = overlap;
    go.tm_out = tm_y; go.accumulate = 1;
    go.gate_mod = mod_l; go.tok_seq = meta + s->ml.tok_seq; go.gate_which = 2;
    go.pair = pair_d;
    go.bn = pair_d ? 256 : gemm_pick_bn(T, d, s->sm_count);
    go.ksplit = pair_d ? 1 : pick_ksplit(T, d, q_dim, go.bn, s->sm_count);
    go.stream_k_slots = pair_d ? gemm_pick_stream_k(T, d, q_dim, s->sm_count) : 0;
    go.tile_turn = reinterpret_cast<int*>(s->ws_dev + s->ws.turn);
    go.status = status;
    go.smid_log = slots(5);
    if (fold_norm) fold_out(go, w.g_mlp);
    if (skinny(q_dim, d, kGemmResid)) {
      SkinnyParams k = skinny_base(o, q_dim, d, kGemmResid);
      k.w[0] = wo.w_o; k.y = x; k.accumulate = 1;
      k.gate_mod = go.gate_mod; k.tok_seq = go.tok_seq; k.gate_which = 2;
      k.smid_log = slots(5);
      if (sk_fold_mlp) sk_fold_out(k, w.g_mlp, skinny(d, F, kGemmGateUp));
      LaunchTimer t(s, 5, stream); where = "out-proj gemm"; e = launch_gemm_skinny(k, sm_budget, stream);
    } else { LaunchTimer t(s, 5, stream); where = "out-proj gemm"; e = launch_gemm(go, sm_budget, stream); }
    if (e != cudaSuccess) break;

    np.x_bf16 = nullptr;
    np.gain = static_cast<const __nv_bfloat16*>(w.g_mlp);
    np.mod_which = 3;
    if (!fold_norm && !sk_fold_mlp) { LaunchTimer t(s, 0, stream); where = "rmsnorm"; e = launch_rmsnorm(np, sm_budget, stream); }
    if (e != cudaSuccess) break;

    GemmParams gu{};
    gu.tm_a = a_rows == 128 ? s->tm_h : s->tm_h_s[a_sel];
    gu.a_box_rows = a_rows;
    gu.tm_b[0] = m.wgate; gu.tm_b[1] = m.wup; gu.tm_b[2] = m.wup;
    gu.M = T; gu.N = F; gu.K = d;
    gu.mode = kGemmGateUp;
    gu.ab_f16 = f16;
    gu.overlap = overlap;
    gu.act_f16 = f16;
    gu.pair = pair_gu;
    gu.tm_act = s->tm_act_st;
    gu.status = status;
    gu.smid_log = slots(6);
    if (fold_norm || sk_fold_mlp) fold_in(gu);
    if (skinny(d, F, kGemmGateUp)) {
      SkinnyParams k = skinny_base(h, d, F, kGemmGateUp);
      k.w[0] = wo.w_gate; k.w[1] = wo.w_up;
      k.act = reinterpret_cast<__nv_bfloat16*>(s->ws_dev + s->ws.act); k.act_f16 = f16;
      k.smid_log = slots(6);
      if (sk_fold_mlp) sk_fold_in(k);
      else k.in_row_rs = gu.in_row_rs;
      LaunchTimer t(s, 6, stream); where = "gate/up gemm"; e = launch_gemm_skinny(k, sm_budget, stream);
    } else { LaunchTimer t(s, 6, stream); where = "gate/up gemm"; e = launch_gemm(gu, sm_budget, stream); }
    if (e != cudaSuccess) break;

    GemmParams gd{};
    gd.tm_a = a_rows == 128 ? s->tm_act : s->tm_act_s[a_sel];
    gd.a_box_rows = a_rows;
    gd.tm_b[0] = m.wdown; gd.tm_b[1] = m.wdown; gd.tm_b[2] = m.wdown;
    gd.M = T; gd.N = d; gd.K = F;
    gd.mode = kGemmResid;
    gd.ab_f16 = f16;
    gd.overlap = overlap;
    gd.tm_out = tm_y; gd.accumulate = 1;
    gd.gate_mod = mod_l; gd.tok_seq = meta + s->ml.tok_seq; gd.gate_which = 5;
    gd.pair = pair_d;
    gd.bn = pair_d ? 256 : gemm_pick_bn(T, d, s->sm_count);
    gd.ksplit = pair_d ? 1 : pick_ksplit(T, d, F, gd.bn, s->sm_count);
    gd.stream_k_slots = pair_d ? gemm_pick_stream_k(T, d, F, s->sm_count) : 0;
    gd.tile_turn = reinterpret_cast<int*>(s->ws_dev + s->ws.turn);
    gd.status = status;
    gd.smid_log = slots(7);
    if (fold_norm && l + 1 < c.n_layers) fold_out(gd, s->layers[l + 1].g_attn);
    if (skinny(F, d, kGemmResid)) {
      SkinnyParams k = skinny_base(s->ws_dev + s->ws.act, F, d, kGemmResid);
      k.w[0] = wo.w_down; k.y = x; k.accumulate = 1;
      k.gate_mod = gd.gate_mod; k.tok_seq = gd.tok_seq; k.gate_which = 5;
      k.smid_log = slots(7);
      if (sk_fold_attn && l + 1 < c.n_layers) sk_fold_out(k, s->layers[l + 1].g_attn, skinny(d, q_dim + 2 * kv_dim, kGemmQkv));
      LaunchTimer t(s, 7, stream); where = "down gemm"; e = launch_gemm_skinny(k, sm_budget, stream);
    } else { LaunchTimer t(s, 7, stream); where = "down gemm"; e = launch_gemm(gd, sm_budget, stream); }
    if (e != cudaSuccess) break;
  }
  return e == cudaSuccess ? HS_OK : cuda_fail(where, e);
}

hs_status_t hs_stage_set_qkv_bias(hs_stage_t* s, int32_t layer, const void* b_q, const void* b_k, const void* b_v) {
  if (!s || layer < 0 || layer >= s->cfg.n_layers) return HS_ERR_INVALID_ARG;
  if (s->cfg.device < 0) return HS_ERR_NO_DEVICE;
  const void* b[3] = {b_q, b_k, b_v};
  for (const void* ptr : b)
    if (reinterpret_cast<uintptr_t>(ptr) & 15) return HS_ERR_INVALID_ARG;
  for (int i = 0; i < 3; ++i) s->qkv_bias[layer].b[i] = static_cast<const __nv_bfloat16*>(b[i]);
  return HS_OK;
}

hs_status_t hs_stage_set_modulation(hs_stage_t* s, const void* mod) {
  if (!s || (reinterpret_cast<uintptr_t>(mod) & 15)) return HS_ERR_INVALID_ARG;
  if (s->cfg.device < 0) return HS_ERR_NO_DEVICE;
  s->modulation = static_cast<const float*>(mod);
  return HS_OK;
}

hs_status_t hs_stage_status(hs_stage_t* s) {
  if (!s) return HS_ERR_INVALID_ARG;
  if (s->cfg.device < 0) return HS_ERR_NO_DEVICE;
  DeviceGuard guard(s->cfg.device);
  int v = 0;
  if (cudaMemcpy(&v, s->ws_dev + s->ws.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return HS_ERR_CUDA;
  return v == 0 ? HS_OK : static_cast<hs_status_t>(v);
}

hs_status_t hs_stage_saturation_count(hs_stage_t* s, int64_t* count) {
  if (!s || !count) return HS_ERR_INVALID_ARG;
  if (s->cfg.device < 0) return HS_ERR_NO_DEVICE;
  DeviceGuard guard(s->cfg.device);
  int v = 0;
  if (cudaMemcpy(&v, s->ws_dev + s->ws.status + 4, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return HS_ERR_CUDA;
  *count = int64_t(uint32_t(v));
  return HS_OK;
}

hs_status_t hs_stage_profile_enable(hs_stage_t* s, int32_t enable) {
  if (!s) return HS_ERR_INVALID_ARG;
  if (s->cfg.device < 0) return HS_ERR_NO_DEVICE;
  s->profile = enable != 0;
  return HS_OK;
}

hs_status_t hs_stage_profile_read(hs_stage_t* s, float* ms, int32_t* launches) {
  if (!s || !ms || !launches) return HS_ERR_INVALID_ARG;
  if (s->cfg.device < 0) return HS_ERR_NO_DEVICE;
  DeviceGuard guard(s->cfg.device);
  hs_status_t st = HS_OK;
  for (const hs_stage::Timed& t : s->timed) {
    float v = 0.f;
    if (cudaEventSynchronize(t.b) != cudaSuccess || cudaEventElapsedTime(&v, t.a, t.b) != cudaSuccess) st = HS_ERR_CUDA;
    if (t.cls >= 0 && t.cls < HS_PROFILE_CLASSES) {
      ms[t.cls] += v;
      launches[t.cls] += 1;
    }
    s->event_pool.push_back(t.a);
    s->event_pool.push_back(t.b);
  }
  s->timed.clear();
  return st;
}

hs_status_t hs_stage_debug_buffer(hs_stage_t* s, const char* name, void** dev_ptr, size_t* bytes) {
  if (!s || !name || !dev_ptr || !bytes) return HS_ERR_INVALID_ARG;
  if (s->cfg.device < 0) return HS_ERR_NO_DEVICE;
  const hs_stage_config_t& c = s->cfg;
  const size_t T = c.max_tokens, q_dim = size_t(c.n_q_heads) * c.head_dim;
  const std::string n(name);
  size_t off, sz;
  if (n == "h") { off = s->ws.h; sz = T * c.d_model * 2; }
  else if (n == "q") { off = s->ws.q; sz = T * q_dim * 2; }
  else if (n == "o") { off = s->ws.o; sz = T * q_dim * 2; }
  else if (n == "act") { off = s->ws.act; sz = T * c.d_ffn * 2; }
  else if (n == "smid") {
    // asking for the census switches it on for the following steps
    s->census = true;
    off = s->ws.smid;
    sz = size_t(HS_PROFILE_CLASSES) * kSmidSlots * 4;
  }
  else return HS_ERR_INVALID_ARG;
  *dev_ptr = s->ws_dev + off;
  *bytes = sz;
  return HS_OK;
}

// Whose-turn words for bare GEMM calls: a zero-initialised array of the library image (device symbols start at zero and
// the kernels leave the words at zero), its device address resolved once per device.
static __device__ int g_op_turn[hs::kGemmTurnWords];
static int* op_turn_words(int dev) {
  static std::mutex m;
  static int* ptr[64] = {};
  if (dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(m);
  if (!ptr[dev]) {
    void* q = nullptr;
    if (cudaGetSymbolAddress(&q, g_op_turn) != cudaSuccess) return nullptr;
    ptr[dev] = static_cast<int*>(q);
  }
  return ptr[dev];
}

static hs_status_t op_gemm(const void* a, const void* w, const float* resid, float* out, int32_t M, int32_t N, int32_t K,
                           int32_t sm_budget, int32_t* status_dev, void* cuda_stream, int ab_f16) {
  if (!a || !w || !out || !status_dev || M < 1 || N < 1 || K < 1) return HS_ERR_INVALID_ARG;
  if ((N & 7) || (K & 7)) return HS_ERR_UNSUPPORTED_SHAPE;
  if ((reinterpret_cast<uintptr_t>(a) & 15) || (reinterpret_cast<uintptr_t>(w) & 15) ||
      (reinterpret_cast<uintptr_t>(out) & 15) || (reinterpret_cast<uintptr_t>(resid) & 15))
    return HS_ERR_INVALID_ARG;
  int dev = 0;
  int sm_count = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || !device_info(dev, &sm_count, &major)) return HS_ERR_CUDA;
  if (major != 10) return HS_ERR_CUDA;
  if (sm_budget < 1 || sm_budget > sm_count) return HS_ERR_INVALID_BUDGET;
  if (ensure_attributes(dev) != HS_OK) return HS_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // the kernels add into `out`: a residual that lives elsewhere is copied there first
  if (resid && resid != out &&
      cudaMemcpyAsync(out, resid, size_t(M) * N * 4, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
    return HS_ERR_CUDA;
  if (gemm_skinny_wins(M, K, N, kGemmResid, 0, sm_count)) {
    SkinnyParams k{};
    k.a = a; k.w[0] = w; k.T = M; k.K = K; k.N = N; k.mode = kGemmResid;
    k.ab_f16 = ab_f16; k.y = out; k.accumulate = resid != nullptr;
    const cudaError_t e = launch_gemm_skinny(k, sm_budget, stream);
    return e == cudaSuccess ? HS_OK : cuda_fail("small-step gemm", e);
  }
  GemmParams g{};
  if (!encode_2d(&g.tm_a, a, M, K, 128) || !encode_2d(&g.tm_b[0], w, N, K, 128) ||
      !encode_2d(&g.tm_out, out, M, N, 32, true))
    return HS_ERR_CUDA;
  g.tm_b[1] = g.tm_b[0];
  g.tm_b[2] = g.tm_b[0];
  g.M = M; g.N = N; g.K = K;
  g.mode = kGemmResid;
  g.ab_f16 = ab_f16;
  g.accumulate = resid != nullptr;
  g.pair = M > 128;
  g.bn = g.pair ? 256 : gemm_pick_bn(M, N, sm_count);
  g.status = status_dev;
  // The ordered adds of the stream-K form need whose-turn words that are zero between launches.  A bare GEMM call has
  // no stage workspace, so it uses a word array of the library image (shared by all bare GEMM calls of the process:
  // such calls must not overlap on the GPU when they take this form; the stage's GEMMs use the stage's own words).
  g.stream_k_slots = g.pair ? gemm_pick_stream_k(M, N, K, sm_count) : 0;
  if (g.stream_k_slots > 0) {
    g.tile_turn = op_turn_words(dev);
    if (!g.tile_turn) g.stream_k_slots = 0;
  }
  const cudaError_t e = launch_gemm(g, sm_budget, stream);
  return e == cudaSuccess ? HS_OK : cuda_fail("gemm", e);
}

hs_status_t hs_op_gemm_bf16(const void* a, const void* w, const float* resid, float* out, int32_t M, int32_t N, int32_t K,
                            int32_t sm_budget, int32_t* status_dev, void* cuda_stream) {
  return op_gemm(a, w, resid, out, M, N, K, sm_budget, status_dev, cuda_stream, 0);
}

hs_status_t hs_op_gemm_f16(const void* a, const void* w, const float* resid, float* out, int32_t M, int32_t N,
                                int32_t K, int32_t sm_budget, int32_t* status_dev, void* cuda_stream) {
  return op_gemm(a, w, resid, out, M, N, K, sm_budget, status_dev, cuda_stream, 1);
}

}  // extern "C"

// ------------------------------------------------------------ ends of the stage --
struct hs_head {
  hs_head_config_t cfg;
  int sm_count = 0;
  uint8_t* ws_dev = nullptr;       // [max_rows][d] bf16 h, then the status word
  size_t off_status = 0;
  const __nv_bfloat16* g_final = nullptr;
  CUtensorMap tm_h, tm_w;
};

namespace {
bool head_config_ok(const hs_head_config_t& c) {
  return c.abi_version == HS_ABI_VERSION && c.device >= 0 && c.d_model >= 64 && c.d_model % 8 == 0 && c.vocab >= 8 &&
         c.vocab % 8 == 0 && c.max_rows >= 1 && c.max_rows <= 128 && c.rms_eps > 0.f;
}
size_t head_status_offset(const hs_head_config_t& c) { return align_up(size_t(c.max_rows) * c.d_model * 2, 1024); }
}  // namespace

size_t hs_head_workspace_bytes(const hs_head_config_t* cfg) {
  if (!cfg || !head_config_ok(*cfg)) return 0;
  return head_status_offset(*cfg) + 1024;
}

hs_status_t hs_head_create(const hs_head_config_t* cfg, const void* g_final, const void* w_vocab, void* workspace_dev,
                           hs_head_t** out) {
  if (!cfg || !out) return HS_ERR_INVALID_ARG;
  *out = nullptr;
  if (!head_config_ok(*cfg)) return cfg->abi_version != HS_ABI_VERSION ? HS_ERR_INVALID_ARG : HS_ERR_UNSUPPORTED_SHAPE;
  if (!g_final || !w_vocab || !workspace_dev) return HS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(g_final) & 15) || (reinterpret_cast<uintptr_t>(w_vocab) & 15) ||
      (reinterpret_cast<uintptr_t>(workspace_dev) & 255))
    return HS_ERR_INVALID_ARG;
  DeviceGuard guard(cfg->device);
  if (!guard.ok) return HS_ERR_CUDA;
  int sm_count = 0, major = 0;
  if (!device_info(cfg->device, &sm_count, &major)) return fail("hs_head_create: device attribute query failed");
  if (major != 10) return fail("hs_head_create: the device is not compute capability 10.x");
  hs_status_t st = ensure_attributes(cfg->device);
  if (st != HS_OK) return st;
  std::unique_ptr<hs_head> h(new (std::nothrow) hs_head());
  if (!h) return HS_ERR_INVALID_ARG;
  h->cfg = *cfg;
  h->sm_count = sm_count;
  h->ws_dev = static_cast<uint8_t*>(workspace_dev);
  h->off_status = head_status_offset(*cfg);
  h->g_final = static_cast<const __nv_bfloat16*>(g_final);
  if (!encode_2d(&h->tm_h, h->ws_dev, cfg->max_rows, cfg->d_model, 128) ||
      !encode_2d(&h->tm_w, w_vocab, cfg->vocab, cfg->d_model, 128))
    return HS_ERR_CUDA;
  if (cudaMemset(h->ws_dev + h->off_status, 0, 256) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess)
    return HS_ERR_CUDA;
  *out = h.release();
  return HS_OK;
}

hs_status_t hs_head_step(hs_head_t* h, const float* y, const int32_t* rows, int32_t n, float* logits, int32_t* tokens,
                         int32_t sm_budget, void* cuda_stream) {
  if (!h || !y || !rows || !logits || !tokens || n < 1 || n > h->cfg.max_rows) return HS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(logits) & 15) return HS_ERR_INVALID_ARG;
  if (sm_budget < 1 || sm_budget > h->sm_count) return HS_ERR_INVALID_BUDGET;
  DeviceGuard guard(h->cfg.device);
  if (!guard.ok) return HS_ERR_CUDA;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int* status = reinterpret_cast<int*>(h->ws_dev + h->off_status);
  const int d = h->cfg.d_model, V = h->cfg.vocab;

  NormParams np{};
  np.x_f32 = y;
  np.gain = h->g_final;
  np.h = reinterpret_cast<__nv_bfloat16*>(h->ws_dev);
  np.T = n;
  np.d = d;
  np.eps = h->cfg.rms_eps;
  np.row_index = rows;
  np.status = status;
  cudaError_t e = launch_rmsnorm(np, sm_budget, stream);
  if (e != cudaSuccess) return cuda_fail("head rmsnorm", e);

  GemmParams g{};
  g.tm_a = h->tm_h;
  g.tm_b[0] = g.tm_b[1] = g.tm_b[2] = h->tm_w;
  if (!encode_2d(&g.tm_out, logits, n, V, 32, true)) return HS_ERR_CUDA;
  g.M = n; g.N = V; g.K = d;
  g.mode = kGemmResid;
  g.accumulate = 0;                          // plain store of the logits
  g.pair = 0;
  g.bn = gemm_pick_bn(n, V, h->sm_count);
  g.ksplit = 1;
  g.status = status;
  e = launch_gemm(g, sm_budget, stream);
  if (e != cudaSuccess) return cuda_fail("head gemm", e);

  ArgmaxParams a{};
  a.logits = logits;
  a.tokens = tokens;
  a.n = n;
  a.vocab = V;
  e = launch_argmax(a, sm_budget, stream);
  return e == cudaSuccess ? HS_OK : cuda_fail("head argmax", e);
}

hs_status_t hs_head_status(hs_head_t* h) {
  if (!h) return HS_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  int v = 0;
  if (cudaMemcpy(&v, h->ws_dev + h->off_status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return HS_ERR_CUDA;
  return v == 0 ? HS_OK : static_cast<hs_status_t>(v);
}

hs_status_t hs_head_destroy(hs_head_t* h) {
  if (!h) return HS_ERR_INVALID_ARG;
  delete h;
  return HS_OK;
}

hs_status_t hs_op_embed(const int32_t* tokens, int32_t n, const void* table, int32_t vocab, int32_t d_model, void* x_out,
                        int32_t sm_budget, int32_t* status_dev, void* cuda_stream) {
  if (!tokens || !table || !x_out || !status_dev || n < 1 || vocab < 1) return HS_ERR_INVALID_ARG;
  if (d_model < 8 || d_model % 8 != 0) return HS_ERR_UNSUPPORTED_SHAPE;
  if ((reinterpret_cast<uintptr_t>(table) & 15) || (reinterpret_cast<uintptr_t>(x_out) & 15)) return HS_ERR_INVALID_ARG;
  int dev = 0;
  int sm_count = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || !device_info(dev, &sm_count, &major)) return HS_ERR_CUDA;
  if (major != 10) return HS_ERR_CUDA;
  if (sm_budget < 1 || sm_budget > sm_count) return HS_ERR_INVALID_BUDGET;
  if (ensure_attributes(dev) != HS_OK) return HS_ERR_CUDA;
  EmbedParams p{};
  p.tokens = tokens;
  p.table = static_cast<const __nv_bfloat16*>(table);
  p.x_out = static_cast<__nv_bfloat16*>(x_out);
  p.n = n;
  p.vocab = vocab;
  p.d = d_model;
  p.status = status_dev;
  const cudaError_t e = launch_embed(p, sm_budget, static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? HS_OK : cuda_fail("embed", e);
}
