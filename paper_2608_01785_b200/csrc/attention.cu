// The decode attention kernel of its own and its launcher (the kernel's body: attention_decode.cuh).
#include "attention_decode.cuh"

namespace hs {
namespace {

template <int DH>
__global__ void __launch_bounds__(DC_THREADS, 1) attn_decode_kernel(const __grid_constant__ AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full_all = reinterpret_cast<uint64_t*>(smem + DC_WARPS * DC_STAGES * 2 * Geom<DH>::PAGE_BYTES);
  log_smid(p.smid_log ? p.smid_log + kSmidSlots : nullptr);
  attn_decode_body<DH>(p, p.layer, p.counters, smem, full_all, int(blockIdx.x), int(gridDim.x), [] {
    griddep_wait();
    griddep_launch_dependents();
  });
}

template <typename K>
cudaError_t set_smem(K kernel, int bytes) {
  return set_kernel_smem(kernel, bytes);
}

}  // namespace

cudaError_t attention_set_attributes() {
  cudaError_t e;
  if ((e = attention_prefill_set_attributes()) != cudaSuccess) return e;
  if ((e = set_smem(attn_decode_kernel<64>, dc_smem_bytes<64>())) != cudaSuccess) return e;
  if ((e = set_smem(attn_decode_kernel<128>, dc_smem_bytes<128>())) != cudaSuccess) return e;
  return cudaSuccess;
}

cudaError_t launch_attention_decode(const AttnParams& p, int sm_budget, cudaStream_t stream) {
  if (p.n_decode_items <= 0) return cudaSuccess;
  const int work = p.decode_group ? p.n_decode_items / DC_WARPS : p.n_decode_items;     // groups, or items
  const int grid = work < sm_budget ? work : sm_budget;
  if (p.head_dim == 128)
    return launch_step_kernel(attn_decode_kernel<128>, grid, DC_THREADS, dc_smem_bytes<128>(), stream, p.overlap != 0, p);
  else
    return launch_step_kernel(attn_decode_kernel<64>, grid, DC_THREADS, dc_smem_bytes<64>(), stream, p.overlap != 0, p);
}

}  // namespace hs
