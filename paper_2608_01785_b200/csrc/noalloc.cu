// hs_op_decode_attention_noalloc: decode attention whose scratch lives inside the library image.
//
// The regular path keeps the decode kernel's scratch (split-KV partials, the work-queue head, the
// step's integer metadata) in a workspace the caller allocates.  Some callers have no way to get one: a
// serving process that handed every free byte of HBM to its KV pool at start-up cannot obtain scratch
// later (the allocation fails, or succeeds only by stalling every stream of the device while the
// driver maps memory), and a plug-in that is handed raw device pointers by a host runtime may simply
// not be allowed to call the allocator.  For them this file carries a fixed scratch area in a
// file-scope __device__ array; the entry point below runs the same decode kernel on it and calls no
// allocating routine: no cudaMalloc / cudaFree / cudaHostAlloc, no heap, no library that allocates.  The
// call's integer metadata is assembled in a fixed host array of the library image (guarded by a mutex).
//
// The array is a device symbol.  In host code its name is only a stand-in, not a device address, so
// the address is obtained once per device with cudaGetSymbolAddress (with that device current) and it
// is that address which the kernels receive.
#include <math.h>
#include <string.h>

#include <mutex>

#include "../../include/horizonserve_ops.h"
#include "hs_internal.h"
#include "kernels.h"

namespace hs {
namespace {

constexpr int kMaxSeqs = HS_NOALLOC_MAX_SEQS;
constexpr int kMaxPagesPerSeq = HS_NOALLOC_MAX_PAGES_PER_SEQ;
constexpr int kMaxItems = HS_NOALLOC_MAX_ITEMS;

// Layout of the scratch area (offsets in 4-byte words).  The integer block is refreshed by every call
// (one host-to-device copy, which also zeroes the queue heads and the status word); the partials are
// fully rewritten for the items of the call before they are read.
constexpr int kOffCounters = 0;                                   // [4]  work-queue heads, must start at 0
constexpr int kOffStatus = 4;                                     // [4]  device status word
constexpr int kOffGroupDone = 8;                                  // [kMaxSeqs * 16] finished splits per group, 0
constexpr int kOffSeqTok0 = kOffGroupDone + kMaxSeqs * 16;        // [kMaxSeqs]
constexpr int kOffSeqCtx = kOffSeqTok0 + kMaxSeqs;                // [kMaxSeqs]
constexpr int kOffTables = kOffSeqCtx + kMaxSeqs;                 // [kMaxSeqs * kMaxPagesPerSeq]
constexpr int kOffItems = kOffTables + kMaxSeqs * kMaxPagesPerSeq;   // [kMaxItems * 8]
constexpr int kOffRows = kOffItems + kMaxItems * 8;               // [kMaxSeqs * 4]
constexpr int kMetaWords = kOffRows + kMaxSeqs * 4;
constexpr int kOffPartMl = (kMetaWords + 63) & ~63;               // [kMaxItems * 16 * 2] floats
constexpr int kOffPartO = kOffPartMl + kMaxItems * 32;            // [kMaxItems * 16 * 128] floats
constexpr int kScratchWords = kOffPartO + kMaxItems * 16 * 128;   // about 4.3 MB in all

// Held by every GPU that loads the library, until the process exits.
static __device__ __align__(256) uint32_t g_noalloc_scratch[kScratchWords];

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// What the first call on a device finds out once and every later call reuses.
struct DeviceSetup {
  uint32_t* scratch = nullptr;   // device address of g_noalloc_scratch on this device
  int sm_count = 0, cc_major = 0;
};
std::mutex g_mutex;              // guards the set-up table, the encode entry point and the host metadata array
DeviceSetup g_setup[64];
EncodeTiledFn g_encode = nullptr;
int32_t g_meta[kMetaWords];      // the call's integer metadata on the host: fixed, shared, filled under g_mutex
int g_last_device = -1;          // device of the most recent call (for hs_op_decode_attention_noalloc_status)

// First use on a device (that device current): resolve the symbol's device address, read the two device
// attributes the argument checks need, raise the kernels' shared-memory limit and fetch the driver's tensor-map
// encoder.  Called with g_mutex held.
hs_status_t setup_device(int dev, const DeviceSetup** out) {
  DeviceSetup& d = g_setup[dev];
  if (!d.scratch) {
    int sm = 0, major = 0;
    if (cudaDeviceGetAttribute(&sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
      return HS_ERR_CUDA;
    if (major != 10) return HS_ERR_CUDA;            // the kernels exist for sm_100a only
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) return HS_ERR_CUDA;
    if (attention_set_attributes() != cudaSuccess) return HS_ERR_CUDA;
    if (!g_encode) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult q;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
          q != cudaDriverEntryPointSuccess)
        return HS_ERR_CUDA;
      g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    d.sm_count = sm;
    d.cc_major = major;
    d.scratch = static_cast<uint32_t*>(ptr);
  }
  *out = &d;
  return HS_OK;
}

bool encode_pool_map(CUtensorMap* m, const void* pool, uint64_t rows, uint64_t head_dim) {
  EncodeTiledFn fn = g_encode;
  cuuint64_t dims[2] = {head_dim, rows};
  cuuint64_t strides[1] = {head_dim * 2};
  cuuint32_t box[2] = {64, 16};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(pool), dims,
            strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace
}  // namespace hs

using namespace hs;

extern "C" hs_status_t hs_op_decode_attention_noalloc(const void* q_dev, const void* kv_pool_dev, int32_t n_layers,
                                                      int32_t layer, int32_t num_pages, int32_t n_q_heads,
                                                      int32_t n_kv_heads, int32_t head_dim, int32_t n_seqs,
                                                      const int32_t* kv_len, const int32_t* block_tables,
                                                      int32_t max_pages_per_seq, void* o_dev, int32_t sm_budget,
                                                      void* cuda_stream) {
  if (!q_dev || !kv_pool_dev || !o_dev || !kv_len || !block_tables) return HS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(q_dev) & 15) || (reinterpret_cast<uintptr_t>(o_dev) & 15) ||
      (reinterpret_cast<uintptr_t>(kv_pool_dev) & 255))
    return HS_ERR_INVALID_ARG;
  if (n_layers < 1 || layer < 0 || layer >= n_layers || num_pages < 1 || n_seqs < 1 || max_pages_per_seq < 1)
    return HS_ERR_INVALID_ARG;
  if ((head_dim != 64 && head_dim != 128) || n_kv_heads < 1 || n_q_heads % n_kv_heads != 0 ||
      n_q_heads / n_kv_heads > 16 || n_kv_heads > 16)
    return HS_ERR_UNSUPPORTED_SHAPE;
  // the fixed scratch area bounds the problem size
  if (n_seqs > kMaxSeqs || max_pages_per_seq > kMaxPagesPerSeq) return HS_ERR_UNSUPPORTED_SHAPE;
  const int64_t pool_rows = int64_t(n_layers) * 2 * num_pages * n_kv_heads * kPage;
  if (pool_rows >= (int64_t(1) << 31)) return HS_ERR_UNSUPPORTED_SHAPE;

  // integer metadata, assembled in the library's fixed host array (no heap, no pinned allocation); the lock is
  // held until the copy below has taken the array's contents
  std::lock_guard<std::mutex> lock(g_mutex);
  int32_t* meta = g_meta;
  memset(meta, 0, sizeof(int32_t) * (kOffSeqTok0));
  int n_items = 0;
  for (int s = 0; s < n_seqs; ++s) {
    const int keys = kv_len[s];
    if (keys < 1) return HS_ERR_INVALID_ARG;
    const int need = ceil_div(keys, kPage);
    if (need > max_pages_per_seq) return HS_ERR_BAD_BLOCK_TABLE;
    for (int i = 0; i < need; ++i) {
      const int32_t pg = block_tables[size_t(s) * max_pages_per_seq + i];
      if (pg < 0 || pg >= num_pages) return HS_ERR_BAD_BLOCK_TABLE;
      meta[kOffTables + s * max_pages_per_seq + i] = pg;
    }
    const int splits = ceil_div(keys, kDecodeSplit);
    if (n_items + n_kv_heads * splits > kMaxItems) return HS_ERR_UNSUPPORTED_SHAPE;
    meta[kOffSeqTok0 + s] = s;           // one query row per sequence
    meta[kOffSeqCtx + s] = keys - 1;
    int32_t* row = meta + kOffRows + s * 4;
    row[0] = s; row[1] = s; row[2] = n_items; row[3] = splits;
    for (int hk = 0; hk < n_kv_heads; ++hk)
      for (int j = 0; j < splits; ++j) {
        int32_t* it = meta + kOffItems + (n_items + hk * splits + j) * 8;
        it[0] = s; it[1] = hk; it[2] = j * kDecodeSplit;
        it[3] = keys < (j + 1) * kDecodeSplit ? keys : (j + 1) * kDecodeSplit;
        it[4] = s; it[5] = s; it[6] = n_items + hk * splits; it[7] = splits | (j << 16);   // one query row per sequence
      }
    n_items += n_kv_heads * splits;
  }

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return HS_ERR_CUDA;
  const DeviceSetup* setup = nullptr;
  hs_status_t st = setup_device(dev, &setup);
  if (st != HS_OK) return st;
  if (sm_budget < 1 || sm_budget > setup->sm_count) return HS_ERR_INVALID_BUDGET;
  uint32_t* scratch = setup->scratch;
  g_last_device = dev;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  AttnParams a{};
  if (!encode_pool_map(&a.tm_kv, kv_pool_dev, uint64_t(pool_rows), uint64_t(head_dim))) return HS_ERR_CUDA;
  // The metadata copy also resets the queue heads and the status word left by the previous call.  The source is
  // ordinary (pageable) host memory: the runtime has taken its contents when the call returns, possibly after
  // waiting for earlier work of the stream.
  if (cudaMemcpyAsync(scratch, meta, sizeof(int32_t) * kMetaWords, cudaMemcpyHostToDevice, stream) != cudaSuccess)
    return HS_ERR_CUDA;
  int32_t* words = reinterpret_cast<int32_t*>(scratch);
  a.q = static_cast<const __nv_bfloat16*>(q_dev);
  a.o = static_cast<__nv_bfloat16*>(o_dev);
  a.n_q_heads = n_q_heads; a.n_kv_heads = n_kv_heads; a.head_dim = head_dim;
  a.num_pages = num_pages; a.max_pages_per_seq = max_pages_per_seq; a.layer = layer;
  a.seq_tok0 = words + kOffSeqTok0;
  a.seq_ctx = words + kOffSeqCtx;
  a.block_tables = words + kOffTables;
  a.prefill_items = nullptr; a.n_prefill_items = 0;
  a.decode_items = words + kOffItems; a.n_decode_items = n_items;
  a.decode_rows = words + kOffRows; a.n_decode_rows = n_seqs;
  a.part_o = reinterpret_cast<float*>(scratch + kOffPartO);
  a.part_ml = reinterpret_cast<float*>(scratch + kOffPartMl);
  a.counters = words + kOffCounters;
  a.group_done = words + kOffGroupDone;
  a.status = words + kOffStatus;
  if (launch_attention_decode(a, sm_budget, stream) != cudaSuccess) return HS_ERR_CUDA;
  return HS_OK;
}

extern "C" hs_status_t hs_op_decode_attention_noalloc_status(int32_t* status_out) {
  if (!status_out) return HS_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_last_device < 0 || !g_setup[g_last_device].scratch) return HS_ERR_INVALID_ARG;   // no call was made yet
  int32_t v = 0;
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return HS_ERR_CUDA;
  if (prev != g_last_device && cudaSetDevice(g_last_device) != cudaSuccess) return HS_ERR_CUDA;
  const cudaError_t e = cudaMemcpy(&v, g_setup[g_last_device].scratch + kOffStatus, 4, cudaMemcpyDeviceToHost);
  if (prev != g_last_device) cudaSetDevice(prev);
  if (e != cudaSuccess) return HS_ERR_CUDA;
  *status_out = v;
  return HS_OK;
}
