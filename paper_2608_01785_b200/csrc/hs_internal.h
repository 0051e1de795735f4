// Internal declarations shared by the host side (allocator, planner, C ABI) and the kernel launchers.
#pragma once
#include <stdint.h>

#include <unordered_map>
#include <vector>

#include "../../include/horizonserve.h"

namespace hs {

constexpr int kPage = HS_PAGE_SIZE;      // tokens per KV page
constexpr int kDecodeSplit = 256;        // run length that sizes the decode item buffers (the planner may pick 128 when the items still fit)
constexpr int kDecodeWarps = 8;            // warps per block of the decode attention kernel (kernels.h: kDecodeKernelWarps)
constexpr int kDecodeSplitMax = 512;     // largest number of keys per item the planner may choose
constexpr int kDecodeTail = 128;         // keys per piece of a sequence's last, incomplete run (the items that end the kernel)
static_assert(kDecodeSplit % 16 == 0 && kDecodeSplitMax / 16 <= 32, "the decode kernel keeps one page id per lane");
constexpr int kPrefillRows = 128;        // (token, query head of one KV head) rows per prefill work item

inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Tokens per prefill work item: the G query heads of one KV head are stacked head-major as rows of the
// 128-row tile (row = head * tokens + token).  A multiple of 8 so that every head's rows start on a
// 1024-byte boundary of the 128-byte-swizzled shared-memory tile.
inline int prefill_tokens_per_item(int G) {
  const int t = (kPrefillRows / G) & ~7;
  return t < 8 ? 8 : t;
}

// ------------------------------------------------------------------ pages --
// LIFO page allocator: pops on a fresh pool give 0, 1, 2, ...; a freed sequence returns its pages in
// reverse order of acquisition.
class PageAllocator {
 public:
  explicit PageAllocator(int num_pages);
  // Grows seq to ceil(total_tokens / kPage) pages.  Returns HS_OK or HS_ERR_OUT_OF_PAGES (unchanged).
  hs_status_t grow(int64_t seq, int total_tokens, const std::vector<int32_t>** table);
  hs_status_t release(int64_t seq);
  int free_pages() const { return static_cast<int>(free_.size()); }

 private:
  std::vector<int32_t> free_;   // stack; back() is popped next
  std::unordered_map<int64_t, std::vector<int32_t>> owned_;
};

// --------------------------------------------------------- step metadata --
// Offsets (in int32 units) of the arrays inside the per-step metadata block that is copied to the
// device once per step.  Fixed at stage creation from the configuration's maxima.
struct MetaLayout {
  int tok_pos, tok_slot, tok_seq;    // [max_tokens]      absolute position / cache slot / sequence index of each new token
  int seq_tok0, seq_ctx, seq_qlen;   // [max_seqs]        first token row, cached tokens, new tokens
  int block_tables;                  // [max_seqs * max_pages_per_seq]
  int prefill_items;                 // [max_prefill_items * 8]  {seq, kv_head, first token, tokens (at most two tiles),
                                     //                           cached tokens, first token row and new tokens of the sequence, 0}
  int decode_items;                  // [max_decode_items * 8]   {decode row, kv_head, first key, end key,
                                     //                           seq, token row, first partial slot of the group,
                                     //                           splits | index within the group << 16}
  int decode_rows;                   // [max_seqs * 4]           {seq, token row, first item, splits}
  int counters;                      // [n_layers * 2]           work-queue heads, zero at step start
  int group_done;                    // [max_seqs * n_kv_heads]  finished decode splits per group, zero
  int grid_bar;                      // [4]                      arrivals at the one-launch small step's grid barriers, zero
  int small_layers;                  // [n_layers * 24]          SmallLayer records (12 pointers each) of the one-launch small step
  int total;                         // int32 words in the block
  int max_prefill_items, max_decode_items;
};
MetaLayout make_meta_layout(const hs_stage_config_t& c);

struct StepPlan {
  int n_tokens = 0, n_seqs = 0;
  int n_prefill_items = 0, n_decode_items = 0, n_decode_rows = 0;
  int decode_group = 0;           // 1: decode items are eight page slices per (sequence, KV head), group-major (see plan_step)
  // work estimates of the two attention kernels (for the split of the SM budget when they run side by side)
  int64_t prefill_blocks = 0;     // 64-key blocks over all prefill items (an item's two tiles share a block)
  int prefill_longest = 0;        // blocks of the longest prefill item
  int64_t decode_kv_bytes = 0;    // K and V bytes the decode items read, one layer
};

// Validates `b` against `c` and, when `meta` is non-NULL, fills the metadata block (layout `ml`).
// `page_stamp` is scratch of num_pages entries used to detect a page named by two sequences; `stamp`
// must be a value not used by an earlier call.  tok_seq (nullable) receives the owning sequence of each
// token.  Returns HS_OK, HS_ERR_INVALID_ARG or HS_ERR_BAD_BLOCK_TABLE.
// Keys per decode work item for this batch: 128, 256, 384 or 512, whichever lets the device's warps finish the items
// in the fewest, shortest rounds (among the sizes whose item count fits max_items).  A function of the batch and of
// the device's SM count only (never of the budget).
int pick_decode_split(const hs_stage_config_t& c, const hs_batch_t& b, int sm_count, int max_items);
hs_status_t plan_step(const hs_stage_config_t& c, const MetaLayout& ml, const hs_batch_t& b, int sm_count,
                      std::vector<int32_t>& page_stamp, int32_t stamp, int32_t* meta, int32_t* tok_seq,
                      StepPlan* plan);

hs_status_t validate_config(const hs_stage_config_t& c);

}  // namespace hs
