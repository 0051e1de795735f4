// Host-only logic of the stage: configuration checks, the page allocator, and the per-step planner
// that turns a batch descriptor into the integer metadata the kernels consume.  Nothing here depends
// on the SM budget, which is what keeps results identical across budgets.
#include <algorithm>
#include <numeric>

#include "hs_internal.h"

namespace hs {

hs_status_t validate_config(const hs_stage_config_t& c) {
  if (c.abi_version != HS_ABI_VERSION || (c.flags & ~(HS_FLAG_BF16_ACTIVATIONS | HS_FLAG_BIDIRECTIONAL)) != 0) return HS_ERR_INVALID_ARG;
  if (c.n_layers < 1 || c.d_model < 64 || c.n_q_heads < 1 || c.n_kv_heads < 1 || c.d_ffn < 64) return HS_ERR_INVALID_ARG;
  if (c.num_pages < 1 || c.max_tokens < 1 || c.max_seqs < 1 || c.max_pages_per_seq < 1 || c.max_position < 1)
    return HS_ERR_INVALID_ARG;
  if (c.max_seqs > c.max_tokens) return HS_ERR_INVALID_ARG;
  if (!(c.rms_eps >= 0.f) || !(c.rope_base > 1.f)) return HS_ERR_INVALID_ARG;
  if (c.page_size != kPage) return HS_ERR_UNSUPPORTED_SHAPE;
  if (c.head_dim != 64 && c.head_dim != 128) return HS_ERR_UNSUPPORTED_SHAPE;
  if (c.n_q_heads % c.n_kv_heads != 0 || c.n_q_heads / c.n_kv_heads > 16) return HS_ERR_UNSUPPORTED_SHAPE;
  // A 128-wide half of a GEMM tile must lie inside one of q / k / v
  if ((c.n_q_heads * c.head_dim) % 128 != 0 || (c.n_kv_heads * c.head_dim) % 128 != 0) return HS_ERR_UNSUPPORTED_SHAPE;
  // 16-byte rows for tiled copies and vector stores
  if (c.d_model % 8 != 0 || c.d_ffn % 8 != 0) return HS_ERR_UNSUPPORTED_SHAPE;
  // total rows of the pool as seen by a tiled copy must fit a 32-bit coordinate
  const int64_t rows = int64_t(c.n_layers) * 2 * c.num_pages * c.n_kv_heads * kPage;
  if (rows >= (int64_t(1) << 31)) return HS_ERR_UNSUPPORTED_SHAPE;
  return HS_OK;
}

// ------------------------------------------------------------------ pages --
PageAllocator::PageAllocator(int num_pages) {
  free_.resize(num_pages);
  for (int i = 0; i < num_pages; ++i) free_[i] = num_pages - 1 - i;
}

hs_status_t PageAllocator::grow(int64_t seq, int total_tokens, const std::vector<int32_t>** table) {
  auto it = owned_.find(seq);
  const int have = it == owned_.end() ? 0 : static_cast<int>(it->second.size());
  const int need = ceil_div(total_tokens, kPage) - have;
  if (need > static_cast<int>(free_.size())) return HS_ERR_OUT_OF_PAGES;
  std::vector<int32_t>& pages = owned_[seq];
  for (int i = 0; i < need; ++i) {
    pages.push_back(free_.back());
    free_.pop_back();
  }
  *table = &pages;
  return HS_OK;
}

hs_status_t PageAllocator::release(int64_t seq) {
  auto it = owned_.find(seq);
  if (it == owned_.end()) return HS_ERR_UNKNOWN_SEQ;
  for (auto p = it->second.rbegin(); p != it->second.rend(); ++p) free_.push_back(*p);
  owned_.erase(it);
  return HS_OK;
}

// --------------------------------------------------------- step metadata --
MetaLayout make_meta_layout(const hs_stage_config_t& c) {
  MetaLayout m{};
  const int G = c.n_q_heads / c.n_kv_heads;
  m.max_prefill_items = c.n_kv_heads * (c.max_tokens / prefill_tokens_per_item(G) + c.max_seqs);
  // a decode sequence of n keys has at most n / kDecodeSplit whole runs and kDecodeSplitMax / kDecodeTail pieces of a
  // last, incomplete one; cached keys are bounded by the pool
  m.max_decode_items = c.n_kv_heads * (c.max_seqs * 2 * (kDecodeSplitMax / kDecodeTail) +
                                       int((int64_t(c.num_pages) * kPage) / kDecodeSplit) + 1);
  int off = 0;
  auto take = [&](int n) {
    int o = off;
    off += (n + 3) & ~3;   // keep every array 16-byte aligned
    return o;
  };
  m.tok_pos = take(c.max_tokens);
  m.tok_slot = take(c.max_tokens);
  m.tok_seq = take(c.max_tokens);
  m.seq_tok0 = take(c.max_seqs);
  m.seq_ctx = take(c.max_seqs);
  m.seq_qlen = take(c.max_seqs);
  m.block_tables = take(c.max_seqs * c.max_pages_per_seq);
  m.prefill_items = take(m.max_prefill_items * 8);
  m.decode_items = take(m.max_decode_items * 8);
  m.decode_rows = take(c.max_seqs * 4);
  m.counters = take(c.n_layers * 2);
  m.group_done = take(c.max_seqs * c.n_kv_heads);
  m.grid_bar = take(4);
  m.small_layers = take(c.n_layers * 24);
  m.total = off;
  return m;
}

int decode_items_of(int keys, int split) { return keys / split + ceil_div(keys % split, kDecodeTail); }

int pick_decode_split(const hs_stage_config_t& c, const hs_batch_t& b, int sm_count, int max_items) {
  // Every warp of the decode kernel works through whole items, longest first.  In units of the time a warp needs for
  // one page an item costs its pages + 8 (queue, record, page ids, first bytes, partial result, its share of the
  // merge), the whole runs are handed out in rounds -- a short last round leaves most warps idle for a whole item --
  // and the pieces of the incomplete runs fill what the last round leaves free, or add rounds of their own:
  //   cost = rounds x (pages per run + 8) + further rounds of pieces x (pages per piece + 8),
  //   rounds = ceil(whole runs / (0.97 x warps of the device)).
  // Measured on B200, 64 sequences of 512..4096 keys, 4 KV heads (model in brackets): 256 keys 72.6 us (72), 384 keys
  // 67.1 (64), 512 keys 77.8 (80); 16 sequences of 300..800 keys: 128 keys 17 us, 256 keys 21 us.
  const int64_t W = int64_t((sm_count > 0 ? sm_count : 148) * kDecodeWarps) * 97 / 100;
  const int piece_cost = kDecodeTail / kPage + 8;
  int best = kDecodeSplit;
  double best_cost = 1e30;
  for (int split = kDecodeTail; split <= kDecodeSplitMax; split += 128) {
    int64_t whole = 0, pieces = 0;
    for (int s = 0; s < b.n_seqs; ++s)
      if (b.q_len[s] == 1) {
        const int keys = b.ctx_len[s] + 1;
        whole += int64_t(c.n_kv_heads) * (keys / split);
        pieces += int64_t(c.n_kv_heads) * ceil_div(keys % split, kDecodeTail);
      }
    if (whole + pieces == 0) return kDecodeSplit;
    if (whole + pieces > max_items) continue;          // (only the smallest size can exceed the buffers)
    const int run_cost = split / kPage + 8;
    const int64_t rounds = (whole + W - 1) / W;
    const int64_t absorbed = (rounds * W - whole) * (run_cost / piece_cost);
    const int64_t left = pieces > absorbed ? pieces - absorbed : 0;
    const double cost = double(rounds * run_cost + (left + W - 1) / W * piece_cost);
    if (cost < best_cost - 1e-9) {
      best_cost = cost;
      best = split;
    }
  }
  return best;
}

hs_status_t plan_step(const hs_stage_config_t& c, const MetaLayout& ml, const hs_batch_t& b, int sm_count,
                      std::vector<int32_t>& page_stamp, int32_t stamp, int32_t* meta, int32_t* tok_seq,
                      StepPlan* plan) {
  if (!b.q_len || !b.ctx_len || !b.block_tables) return HS_ERR_INVALID_ARG;
  if (b.n_seqs < 1 || b.n_seqs > c.max_seqs || b.n_tokens < 1 || b.n_tokens > c.max_tokens) return HS_ERR_INVALID_ARG;
  const int mpps = c.max_pages_per_seq;
  int64_t total = 0;
  for (int s = 0; s < b.n_seqs; ++s) {
    if (b.q_len[s] < 1 || b.ctx_len[s] < 0) return HS_ERR_INVALID_ARG;
    if (int64_t(b.ctx_len[s]) + b.q_len[s] > c.max_position) return HS_ERR_INVALID_ARG;
    total += b.q_len[s];
  }
  if (total != b.n_tokens) return HS_ERR_INVALID_ARG;
  // block tables: enough pages, ids in range, no page named twice in this step
  for (int s = 0; s < b.n_seqs; ++s) {
    const int need = ceil_div(b.ctx_len[s] + b.q_len[s], kPage);
    if (need > mpps) return HS_ERR_BAD_BLOCK_TABLE;
    for (int i = 0; i < need; ++i) {
      const int32_t pg = b.block_tables[size_t(s) * mpps + i];
      if (pg < 0 || pg >= c.num_pages) return HS_ERR_BAD_BLOCK_TABLE;
      if (page_stamp[pg] == stamp) return HS_ERR_BAD_BLOCK_TABLE;
      page_stamp[pg] = stamp;
    }
  }

  const int G = c.n_q_heads / c.n_kv_heads;
  const int Mt = prefill_tokens_per_item(G);
  const int split = pick_decode_split(c, b, sm_count, ml.max_decode_items);
  // Group mode of the decode attention: when even the smallest run length leaves warps idle (the batch is small) and
  // every (sequence, KV head) group can have a block of its own, a group's pages are dealt evenly to the eight warps
  // of one block, whose partial results then meet in shared memory -- no partials in global memory, no counter, no
  // merging warp.  A function of the batch and the device's SM count, never of the budget.
  bool group_mode = split == kDecodeTail;
  {
    int groups = 0, longest = 0;
    for (int s = 0; s < b.n_seqs; ++s)
      if (b.q_len[s] == 1) { groups += c.n_kv_heads; longest = std::max(longest, b.ctx_len[s] + 1); }
    const int sms = sm_count > 0 ? sm_count : 148;
    if (groups == 0 || groups > sms || longest > kDecodeWarps * 32 * kPage) group_mode = false;
  }
  StepPlan p;
  p.n_tokens = b.n_tokens;
  p.n_seqs = b.n_seqs;

  struct Item { int32_t v[8]; int32_t cost; };
  std::vector<Item> pre;
  struct DecItem { int32_t v[8]; int32_t keys; };
  std::vector<DecItem> dec;
  int n_dec_items = 0, n_dec_rows = 0;
  int t = 0;
  for (int s = 0; s < b.n_seqs; ++s) {
    const int n = b.q_len[s], ctx = b.ctx_len[s];
    if (meta) {
      meta[ml.seq_tok0 + s] = t;
      meta[ml.seq_ctx + s] = ctx;
      meta[ml.seq_qlen + s] = n;
      for (int i = 0; i < mpps; ++i) meta[ml.block_tables + s * mpps + i] = b.block_tables[size_t(s) * mpps + i];
    }
    for (int j = 0; j < n; ++j) {
      const int pos = ctx + j;
      const int slot = b.block_tables[size_t(s) * mpps + pos / kPage] * kPage + pos % kPage;
      if (meta) {
        meta[ml.tok_pos + t + j] = pos;
        meta[ml.tok_slot + t + j] = slot;
        meta[ml.tok_seq + t + j] = s;
      }
      if (tok_seq) tok_seq[t + j] = s;
    }
    if (n == 1 && group_mode) {
      // decode, group mode: eight slices of the sequence's pages per KV head (the last ones may be empty)
      const int keys = ctx + 1, pages = ceil_div(keys, kPage), per = ceil_div(pages, kDecodeWarps) * kPage;
      if (meta) {
        int32_t* row = meta + ml.decode_rows + n_dec_rows * 4;
        row[0] = s; row[1] = t; row[2] = n_dec_items; row[3] = kDecodeWarps;
      }
      for (int hk = 0; hk < c.n_kv_heads; ++hk)
        for (int w = 0; w < kDecodeWarps; ++w) {
          const int k0 = std::min(keys, w * per), k1 = std::min(keys, (w + 1) * per);
          dec.push_back(DecItem{{n_dec_rows, hk, k0, k1, s, t, 0, 1}, 0});
        }
      n_dec_items += c.n_kv_heads * kDecodeWarps;
      p.decode_kv_bytes += int64_t(keys) * 2 * c.n_kv_heads * c.head_dim * 2;
      ++n_dec_rows;
    } else if (n == 1) {
      // decode: keys 0..ctx cut into whole runs of `split` keys and the rest into pieces of kDecodeTail keys; the items
      // of a (sequence, KV head) group keep consecutive partial-result slots in key order, whatever the order the
      // queue hands them out in
      const int keys = ctx + 1, small = kDecodeTail;
      const int n_big = keys / split;
      const int splits = decode_items_of(keys, split);
      if (splits > 0x7fff) return HS_ERR_INVALID_ARG;      // the item record keeps the index within the group in 15 bits
      if (meta) {
        int32_t* row = meta + ml.decode_rows + n_dec_rows * 4;
        row[0] = s; row[1] = t; row[2] = n_dec_items; row[3] = splits;
      }
      for (int hk = 0; hk < c.n_kv_heads; ++hk)
        for (int j = 0; j < splits; ++j) {
          const int k0 = j < n_big ? j * split : n_big * split + (j - n_big) * small;
          const int k1 = j < n_big ? k0 + split : std::min(keys, k0 + small);
          dec.push_back(DecItem{{n_dec_rows, hk, k0, k1, s, t, n_dec_items + hk * splits, splits | (j << 16)}, k1 - k0});
        }
      n_dec_items += c.n_kv_heads * splits;
      p.decode_kv_bytes += int64_t(keys) * 2 * c.n_kv_heads * c.head_dim * 2;
      ++n_dec_rows;
    } else {
      // a prefill item covers two Q tiles of Mt tokens each (the second one may be short or absent)
      for (int t0 = 0; t0 < n; t0 += 2 * Mt)
        for (int hk = 0; hk < c.n_kv_heads; ++hk) {
          const int nt = std::min(2 * Mt, n - t0);
          pre.push_back(Item{{s, hk, t0, nt, ctx, t, n, 0}, ctx + t0 + nt});
          const int keys_item = (c.flags & HS_FLAG_BIDIRECTIONAL) ? ctx + n : ctx + t0 + nt;
          const int blocks = ceil_div(keys_item, 64);
          p.prefill_blocks += blocks;
          p.prefill_longest = std::max(p.prefill_longest, blocks);
        }
    }
    t += n;
  }
  if (int(pre.size()) > ml.max_prefill_items || n_dec_items > ml.max_decode_items) return HS_ERR_INVALID_ARG;
  // longest first, so that the dynamic queue finishes evenly; ties keep batch order
  std::stable_sort(pre.begin(), pre.end(), [](const Item& a, const Item& b2) { return a.cost > b2.cost; });
  // decode items likewise: the long runs first, the short ones fill the end of the kernel
  if (!group_mode) std::stable_sort(dec.begin(), dec.end(), [](const DecItem& a, const DecItem& b2) { return a.keys > b2.keys; });
  if (meta) {
    for (size_t i = 0; i < dec.size(); ++i)
      for (int k = 0; k < 8; ++k) meta[ml.decode_items + int(i) * 8 + k] = dec[i].v[k];
    for (size_t i = 0; i < pre.size(); ++i)
      for (int k = 0; k < 8; ++k) meta[ml.prefill_items + int(i) * 8 + k] = pre[i].v[k];
    for (int i = 0; i < c.n_layers * 2; ++i) meta[ml.counters + i] = 0;
    for (int i = 0; i < c.max_seqs * c.n_kv_heads; ++i) meta[ml.group_done + i] = 0;
    for (int i = 0; i < 4; ++i) meta[ml.grid_bar + i] = 0;
  }
  p.n_prefill_items = int(pre.size());
  p.n_decode_items = n_dec_items;
  p.decode_group = group_mode && n_dec_items > 0 ? 1 : 0;
  p.n_decode_rows = n_dec_rows;
  if (plan) *plan = p;
  return HS_OK;
}

}  // namespace hs
