"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every declared symbol, and its
host logic (page allocator, batch validation, per-token metadata) agrees bit for bit with the
independently written oracle in oracle/paging.py."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle.paging import OutOfPages, PageAllocator, block_table_array, plan_tokens
from paper_2608_01785_b200 import binding as B
from paper_2608_01785_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def host_stage(dims=wl.DIMS["c1_tiny"], num_pages=64, max_tokens=256, max_seqs=16, mpps=8, max_position=128):
    cfg = B.make_config(dims, num_pages, max_tokens, max_seqs, mpps, max_position, device=-1)
    return B.hs_stage_create(cfg, None, 0, 0), cfg


def declared_functions():
    names = []
    for header in ("horizonserve.h", "horizonserve_ops.h", "horizonserve_control.h", "horizonserve_head.h"):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(hs_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_library_loads_and_exports_every_declared_symbol():
    lib = B.lib()
    names = declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(B.EXPORTS)
    assert B.status_str(B.HS_OK) == "HS_OK" and B.status_str(B.HS_ERR_TIMEOUT) == "HS_ERR_TIMEOUT"


def test_step_refuses_to_run_without_a_device():
    stage, cfg = host_stage()
    try:
        batch = B.Batch([1], [0], np.zeros((1, 8), dtype=np.int32), 16, 16)
        with pytest.raises(B.HsError) as e:
            B.hs_stage_step(stage, batch, 8)
        assert e.value.status == B.HS_ERR_NO_DEVICE
        assert B.hs_stage_sm_count(stage) == 0
    finally:
        B.hs_stage_destroy(stage)


def test_config_validation():
    good = wl.DIMS["c1_tiny"]
    assert B.hs_kv_pool_bytes(B.make_config(good, 13, 128, 8, 8, 128, -1)) == 1 * 2 * 13 * 2 * 16 * 64 * 2
    assert B.hs_workspace_bytes(B.make_config(good, 13, 128, 8, 8, 128, -1)) > 0
    bad = [
        wl.StageDims(1, 256, 4, 2, 96, 688),      # head_dim not 64 / 128
        wl.StageDims(1, 256, 5, 2, 64, 688),      # Hq % Hkv
        wl.StageDims(1, 256, 4, 1, 64, 688),      # Hkv * Dh not a multiple of 128
        wl.StageDims(1, 252, 4, 2, 64, 688),      # d % 8
        wl.StageDims(1, 256, 4, 2, 64, 688, page_size=32),
        wl.StageDims(0, 256, 4, 2, 64, 688),
    ]
    for dims in bad:
        cfg = B.make_config(dims, 13, 128, 8, 8, 128, -1)
        assert B.hs_kv_pool_bytes(cfg) == 0 and B.hs_workspace_bytes(cfg) == 0, dims
        with pytest.raises(B.HsError):
            B.hs_stage_create(cfg, None, 0, 0)
    cfg = B.make_config(good, 13, 128, 8, 8, 128, -1)
    cfg.abi_version = 99
    with pytest.raises(B.HsError) as e:
        B.hs_stage_create(cfg, None, 0, 0)
    assert e.value.status == B.HS_ERR_INVALID_ARG


def test_activation_format_flag_sizes_the_workspace():
    """The default stage keeps fp16 copies of the seven projection matrices of every layer in its workspace;
    HS_FLAG_BF16_ACTIVATIONS drops them.  Any other flag bit is refused."""
    dims = wl.DIMS["c1_tiny"]
    cfg16 = B.make_config(dims, 64, 128, 8, 8, 256, device=-1)
    cfgbf = B.make_config(dims, 64, 128, 8, 8, 256, device=-1, flags=B.HS_FLAG_BF16_ACTIVATIONS)
    w_bytes = 2 * dims.n_layers * (2 * dims.q_dim * dims.d_model + 2 * dims.kv_dim * dims.d_model +
                                   3 * dims.d_ffn * dims.d_model)
    extra = B.hs_workspace_bytes(cfg16) - B.hs_workspace_bytes(cfgbf)
    assert w_bytes <= extra <= w_bytes + 7 * 1024 * dims.n_layers
    assert B.hs_kv_pool_bytes(cfg16) == B.hs_kv_pool_bytes(cfgbf) > 0
    bidir = B.make_config(dims, 64, 128, 8, 8, 256, device=-1, flags=B.HS_FLAG_BIDIRECTIONAL)
    assert B.hs_workspace_bytes(bidir) == B.hs_workspace_bytes(cfg16)      # the mask changes no buffer
    bad = B.make_config(dims, 64, 128, 8, 8, 256, device=-1, flags=4)
    assert B.hs_workspace_bytes(bad) == 0 and B.hs_kv_pool_bytes(bad) == 0


def test_allocator_config_1_block_tables_by_hand():
    # sequences allocated in order with 32, 48, 40 + 1 and 64 + 1 tokens; pops yield 0, 1, 2, ...
    stage, _ = host_stage()
    try:
        tables = [B.hs_kv_alloc(stage, s, t, 8) for s, t in enumerate([32, 48, 41, 65])]
        assert tables == [[0, 1], [2, 3, 4], [5, 6, 7], [8, 9, 10, 11, 12]]
        assert B.hs_kv_free_pages(stage) == 64 - 13
    finally:
        B.hs_stage_destroy(stage)


def test_allocator_matches_oracle_under_random_grow_and_free():
    num_pages = 40
    stage, _ = host_stage(num_pages=num_pages, mpps=12)
    ora = PageAllocator(num_pages, 16)
    r = np.random.default_rng(0)
    lens = {}
    try:
        for step in range(400):
            seq = int(r.integers(0, 9))
            if seq in lens and r.random() < 0.3:
                B.hs_kv_free(stage, seq)
                ora.release(seq)
                del lens[seq]
                continue
            total = lens.get(seq, 0) + int(r.integers(0, 40))
            total = min(total, 12 * 16)
            try:
                want = ora.alloc(seq, total)
            except OutOfPages:
                with pytest.raises(B.HsError) as e:
                    B.hs_kv_alloc(stage, seq, total, 12)
                assert e.value.status == B.HS_ERR_OUT_OF_PAGES
                continue
            got = B.hs_kv_alloc(stage, seq, total, 12)
            assert got == want, (step, seq, total)
            lens[seq] = total
            assert B.hs_kv_free_pages(stage) == len(ora.free)
        with pytest.raises(B.HsError) as e:
            B.hs_kv_free(stage, 12345)
        assert e.value.status == B.HS_ERR_UNKNOWN_SEQ
    finally:
        B.hs_stage_destroy(stage)


@pytest.mark.parametrize("name", ["c1_tiny", "c2_shared", "c3_7b", "c4_talker"])
def test_plan_matches_oracle_token_metadata(name):
    dims = wl.DIMS[name]
    batch = wl.make_batch(name, seed=2)
    need = wl.pages_needed(batch)
    mpps = max(-(-t // 16) for t in batch.total_len()) + 1
    cfg = B.make_config(dims, need + 7, batch.n_tokens, batch.n_seqs, mpps, max(batch.total_len()), device=-1)
    stage = B.hs_stage_create(cfg, None, 0, 0)
    try:
        # shuffle the free list first so that page ids are not the identity
        warm = [B.hs_kv_alloc(stage, 1000 + i, 16 * (1 + i % 3), mpps) for i in range(3)]
        for i in (1, 0, 2):
            B.hs_kv_free(stage, 1000 + i)
        ora = PageAllocator(need + 7, 16)
        for i in range(3):
            ora.alloc(1000 + i, 16 * (1 + i % 3))
        for i in (1, 0, 2):
            ora.release(1000 + i)
        tables = [B.hs_kv_alloc(stage, s, t, mpps) for s, t in enumerate(batch.total_len())]
        assert tables == [ora.alloc(s, t) for s, t in enumerate(batch.total_len())]
        bt = block_table_array(tables, mpps)
        seq, pos, slot = B.hs_stage_plan(stage, B.Batch(batch.q_len, batch.ctx_len, bt))
        wseq, wpos, wslot = plan_tokens(batch.q_len, batch.ctx_len, bt, 16)
        assert np.array_equal(seq, wseq) and np.array_equal(pos, wpos) and np.array_equal(slot, wslot)
    finally:
        B.hs_stage_destroy(stage)


def test_plan_rejects_malformed_batches():
    stage, cfg = host_stage(num_pages=16, max_tokens=64, max_seqs=4, mpps=4, max_position=64)
    bt = np.array([[0, 1, -1, -1], [2, -1, -1, -1]], dtype=np.int32)

    def status_of(q_len, ctx_len, tables, n_tokens=None):
        b = B.Batch(q_len, ctx_len, tables)
        if n_tokens is not None:
            b.c.n_tokens = n_tokens
        try:
            B.hs_stage_plan(stage, b)
            return B.HS_OK
        except B.HsError as e:
            return e.status

    try:
        assert status_of([20, 1], [0, 5], bt) == B.HS_OK
        assert status_of([20, 1], [0, 5], bt, n_tokens=20) == B.HS_ERR_INVALID_ARG     # n_tokens != sum q_len
        assert status_of([0, 1], [0, 5], bt) == B.HS_ERR_INVALID_ARG                    # q_len < 1
        assert status_of([20, 1], [0, -1], bt) == B.HS_ERR_INVALID_ARG                  # ctx_len < 0
        assert status_of([20, 1], [50, 5], bt) == B.HS_ERR_INVALID_ARG                  # past max_position
        assert status_of([33, 1], [0, 5], bt) == B.HS_ERR_BAD_BLOCK_TABLE               # needs a 3rd page, has -1
        bad = bt.copy(); bad[1, 0] = 16
        assert status_of([20, 1], [0, 5], bad) == B.HS_ERR_BAD_BLOCK_TABLE              # page id out of range
        dup = bt.copy(); dup[1, 0] = 1
        assert status_of([20, 1], [0, 5], dup) == B.HS_ERR_BAD_BLOCK_TABLE              # page shared by two sequences
        assert status_of([1] * 5, [0] * 5, np.zeros((5, 4), dtype=np.int32)) == B.HS_ERR_INVALID_ARG   # > max_seqs
        assert status_of([65], [0], np.array([[0, 1, 2, 3]], dtype=np.int32)) == B.HS_ERR_INVALID_ARG  # > max_tokens
        # an unused entry beyond the needed pages is not examined
        loose = bt.copy(); loose[0, 3] = 999
        assert status_of([20, 1], [0, 5], loose) == B.HS_OK
    finally:
        B.hs_stage_destroy(stage)


def test_kv_alloc_argument_errors_change_nothing():
    stage, _ = host_stage(num_pages=4, mpps=4)
    try:
        with pytest.raises(B.HsError) as e:
            B.hs_kv_alloc(stage, 0, 5 * 16, 4)           # cap too small for the request
        assert e.value.status == B.HS_ERR_INVALID_ARG
        with pytest.raises(B.HsError) as e:
            B.hs_kv_alloc(stage, 0, 80, 8)               # pool too small
        assert e.value.status == B.HS_ERR_OUT_OF_PAGES
        assert B.hs_kv_free_pages(stage) == 4
        assert B.hs_kv_alloc(stage, 0, 33, 4) == [0, 1, 2]
        assert B.hs_kv_alloc(stage, 0, 20, 4) == [0, 1, 2]   # never shrinks
    finally:
        B.hs_stage_destroy(stage)
