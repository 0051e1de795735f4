"""CPU-only checks of the planner's attention work lists and of the skewed K split (host logic behind the kernels'
work decomposition): every key of every decode sequence is covered exactly once per KV head, the queue order is
longest first, partial slots follow key order, group mode is chosen for small batches only; prefill items cover every
new token once per KV head; the K splits tile the K range without gaps or empty splits."""
import numpy as np
import pytest

from paper_2608_01785_b200 import binding as B
from paper_2608_01785_b200 import workloads as wl


def _stage_and_batch(dims, q_len, ctx_len):
    batch = wl.BatchSpec(list(q_len), list(ctx_len))
    num_pages = wl.pages_needed(batch) + 4
    mpps = max(-(-t // 16) for t in batch.total_len())
    cfg = B.make_config(dims, num_pages, batch.n_tokens, batch.n_seqs, mpps, max(batch.total_len()), device=-1)
    stage = B.hs_stage_create(cfg, None, 0, 0)
    tables = np.full((batch.n_seqs, mpps), -1, dtype=np.int32)
    for s, t in enumerate(batch.total_len()):
        pages = B.hs_kv_alloc(stage, s, t, mpps)
        tables[s, : len(pages)] = pages
    return stage, B.Batch(batch.q_len, batch.ctx_len, tables, 16, 16), batch


def _check_decode(dims, batch, items, group):
    dec_rows = [(s, c) for s, (q, c) in enumerate(zip(batch.q_len, batch.ctx_len)) if q == 1]
    cover = {(s, hk): np.zeros(c + 1, dtype=np.int32) for s, c in dec_rows for hk in range(dims.n_kv_heads)}
    for it in items:
        drow, hk, k0, k1, seq, tok = (int(v) for v in it[:6])
        assert dec_rows[drow][0] == seq and 0 <= hk < dims.n_kv_heads
        assert 0 <= k0 <= k1 <= dec_rows[drow][1] + 1 and (k0 % 16 == 0 or k0 == k1) and k1 - k0 <= 512
        assert group or k1 > k0
        cover[(seq, hk)][k0:k1] += 1
    for c in cover.values():
        assert np.all(c == 1)                      # every key exactly once per KV head
    if group:
        assert len(items) == 8 * len(cover)
        for g in range(len(cover)):                # a group's eight slices are consecutive and in key order
            blk = items[8 * g: 8 * g + 8]
            assert len({(int(r[4]), int(r[1])) for r in blk}) == 1
            assert all(int(blk[w][3]) == int(blk[w + 1][2]) for w in range(7)) and int(blk[0][2]) == 0
    else:
        keys = items[:, 3] - items[:, 2]
        assert np.all(keys[:-1] >= keys[1:])       # the queue hands the items out longest first
        slots = {}
        for it in items:                           # partial slots of a group: consecutive, in key order
            first, splits, idx = int(it[6]), int(it[7]) & 0xffff, int(it[7]) >> 16
            slots.setdefault((int(it[4]), int(it[1])), []).append((int(it[2]), first + idx, first, splits))
        used = []
        for lst in slots.values():
            lst.sort()
            assert len({(f, n) for _, _, f, n in lst}) == 1 and lst[0][3] == len(lst)
            assert [s for _, s, _, _ in lst] == list(range(lst[0][2], lst[0][2] + len(lst)))
            used += [s for _, s, _, _ in lst]
        assert sorted(used) == list(range(len(items)))     # no two groups share a slot


CASES = {
    "talker": ("c4_talker", None),
    "c2": ("c2_shared", None),
    "c3": ("c3_7b", None),
    "one_long": ("c3_7b", ([1], [16000])),
    "many_short": ("c4_talker", ([1] * 200, [3 + 7 * i for i in range(200)])),
    "mixed_runs": ("c3_7b", ([1] * 64 + [300], [127, 128, 129, 255, 256, 257, 383, 384, 385, 511, 512, 513] * 5 + [4000] * 4 + [0])),
}


@pytest.mark.parametrize("name", sorted(CASES))
def test_attention_work_lists_cover_every_key_and_token_once(name):
    wname, custom = CASES[name]
    dims = wl.DIMS[wname]
    if custom is None:
        b0 = wl.make_batch(wname, {"c4_talker": 3, "c2_shared": 1, "c3_7b": 2}[wname])
        q_len, ctx_len = b0.q_len, b0.ctx_len
    else:
        q_len, ctx_len = custom
    stage, batch_c, batch = _stage_and_batch(dims, q_len, ctx_len)
    try:
        dec, group, pre = B.hs_stage_plan_attention(stage, batch_c)
        _check_decode(dims, batch, dec, group)
        # group mode only where every group can have a block (148 SMs without a device) and no slice exceeds 32 pages
        n_groups = sum(1 for q in batch.q_len if q == 1) * dims.n_kv_heads
        if group:
            assert n_groups <= 148 and max(c + 1 for q, c in zip(batch.q_len, batch.ctx_len) if q == 1) <= 4096
        if name in ("c3", "one_long", "many_short"):
            assert not group
        if name in ("talker", "c2"):
            assert group
        # prefill items: every new token of a prefill sequence once per KV head, at most two tiles, longest first
        G = dims.n_q_heads // dims.n_kv_heads
        mt = max(8, (128 // G) & ~7)
        seen = {(s, hk): np.zeros(q, dtype=np.int32) for s, q in enumerate(batch.q_len) if q > 1 for hk in range(dims.n_kv_heads)}
        tok0 = np.concatenate([[0], np.cumsum(batch.q_len)[:-1]])
        for it in pre:
            s, hk, t0, nt, ctx, row0, qn = (int(v) for v in it[:7])
            assert 1 <= nt <= 2 * mt and ctx == batch.ctx_len[s] and qn == batch.q_len[s] and row0 == tok0[s]
            seen[(s, hk)][t0: t0 + nt] += 1
        for c in seen.values():
            assert np.all(c == 1)
        cost = [int(it[4]) + int(it[2]) + int(it[3]) for it in pre]
        assert cost == sorted(cost, reverse=True)
    finally:
        B.hs_stage_destroy(stage)


def test_k_splits_tile_the_k_range():
    for k_blocks in list(range(1, 70)) + [112, 148, 296, 1000]:
        for ks in range(1, 9):
            b = [B.hs_op_gemm_split_begin(k_blocks, ks, i) for i in range(ks + 1)]
            assert b[0] == 0 and b[-1] == k_blocks and all(x <= y for x, y in zip(b, b[1:]))
            lens = [y - x for x, y in zip(b, b[1:])]
            if k_blocks >= 10 * ks * (ks - 1) // 2 + 10 * ks and ks > 1:
                # long enough for the skew: each split ten blocks longer than the one before, the last takes the remainder
                assert all(lens[i + 1] - lens[i] == 10 for i in range(ks - 2)) and lens[-1] - lens[-2] >= 10
                assert min(lens) >= 10
            else:
                assert max(lens) - min(l for l in lens if l > 0) <= max(lens)      # equal runs (the tail may be short or empty)
                assert lens == sorted(lens, reverse=True)
    assert B.hs_op_gemm_split_begin(0, 1, 0) == -1 and B.hs_op_gemm_split_begin(10, 0, 0) == -1
    assert B.hs_op_gemm_split_begin(10, 2, 3) == -1
    # the down-projection of a 64-row step at 7B dimensions: 296 K blocks in 5 splits
    assert [B.hs_op_gemm_split_begin(296, 5, i) for i in range(6)] == [0, 39, 88, 147, 216, 296]
