"""hs_op_decode_attention_noalloc: the decode-attention variant for callers that cannot allocate device
memory (all HBM already given to the KV pool, or a component that only ever receives pointers).  Its
scratch is a fixed array inside the library, shared by every call, so the checks are: the same result as
the regular path (the decode attention inside hs_stage_step, read back through the stage's "o" buffer) and
as the CPU oracle's attention of the same queries over the same cache, on two different calls in a row --
the second one must not see anything the first one left behind -- also when the two calls follow each
other on one stream with no synchronisation in between, and a clear refusal of problems larger than the
fixed scratch.

Collected last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from oracle.oracle import Oracle
from paper_2608_01785_b200 import binding as B
from paper_2608_01785_b200 import workloads as wl
from tests.helpers import make_case, rel_err

TOL = 2e-2


def test_sizes_beyond_the_fixed_scratch_are_refused():
    """Host-side checks come first, so this needs no GPU: nothing is launched for an oversized problem."""
    ok_ptr = 1024   # never dereferenced: the call is refused before any CUDA work

    def status(n_seqs=1, mpps=8, kv=1, hkv=2):
        tables = np.zeros((n_seqs, mpps), dtype=np.int32)
        try:
            B.hs_op_decode_attention_noalloc(ok_ptr, ok_ptr, 1, 0, 4096, 8, hkv, 64, [kv] * n_seqs, tables, ok_ptr, 8)
        except B.HsError as e:
            return e.status
        return B.HS_OK

    assert status(n_seqs=65) == B.HS_ERR_UNSUPPORTED_SHAPE            # more sequences than HS_NOALLOC_MAX_SEQS
    assert status(mpps=257) == B.HS_ERR_UNSUPPORTED_SHAPE             # longer block tables than the scratch holds
    assert status(n_seqs=64, mpps=256, kv=4096, hkv=2) == B.HS_ERR_UNSUPPORTED_SHAPE   # 64*2*16 items > 512
    assert status(kv=0) == B.HS_ERR_INVALID_ARG
    assert status(kv=200, mpps=8) == B.HS_ERR_BAD_BLOCK_TABLE         # needs 13 pages, table has 8


def _decode_case(dims, ctx_len, seed):
    batch = wl.BatchSpec([1] * len(ctx_len), list(ctx_len))
    return make_case(dims, batch, seed=seed, kv_fill=True)


def _oracle_attention(orc, case, dims, q, pool_bits, kv_len):
    """o[s, head] = attention of query row s over keys 0 .. kv_len[s] - 1 of the cache, by the oracle."""
    want = np.zeros((len(kv_len), dims.n_q_heads, dims.head_dim), dtype=np.float32)
    qv = q.reshape(len(kv_len), dims.n_q_heads, dims.head_dim)
    for s, n in enumerate(kv_len):
        for hq in range(dims.n_q_heads):
            want[s, hq], _ = orc.attend(case.cfg, pool_bits, 0, case.block_tables[s], n - 1, hq, qv[s, hq])
    return want.reshape(len(kv_len), -1)


@pytest.mark.gpu
def test_noalloc_decode_attention_matches_the_stage_path_twice_in_a_row():
    from tests.gpu_helpers import make_stage, run_step
    dev = torch.device("cuda:0")
    orc = Oracle("f32")
    problems = [
        (wl.StageDims(1, 512, 8, 2, 64, 1024), [700, 33, 255, 256, 1023, 5, 64, 300], 31),
        (wl.StageDims(1, 512, 8, 1, 128, 1024), [40, 1500, 511, 17], 32),   # other head size, fewer and longer
    ]
    kept = []
    for dims, ctx, seed in problems:
        case = _decode_case(dims, ctx, seed)
        st = make_stage(case, flags=B.HS_FLAG_BF16_ACTIVATIONS)   # the stage's o in bf16, as this call writes it
        try:
            _, pool_bits = run_step(st, case, 148)
            n = case.batch.n_seqs
            q = st.debug_tensor("q")[:n].contiguous()            # queries after RoPE, as the stage used them
            o_stage = st.debug_tensor("o")[:n].float().cpu().numpy()
            o_got = torch.full((n, dims.q_dim), float("nan"), dtype=torch.bfloat16, device=dev)
            kv_len = [c + 1 for c in ctx]                          # the step cached the new token as well
            args = (q.data_ptr(), st.kv_pool.data_ptr(), dims.n_layers, 0, case.cfg.num_pages, dims.n_q_heads,
                    dims.n_kv_heads, dims.head_dim, kv_len, case.block_tables)
            B.hs_op_decode_attention_noalloc(*args, o_got.data_ptr(), 148)
            torch.cuda.synchronize()
            assert B.hs_op_decode_attention_noalloc_status() == B.HS_OK
            got = o_got.float().cpu().numpy()
            assert np.all(np.isfinite(got))
            # against the existing entry point (the stage sizes its split-KV items by batch -- or deals a group's pages
            # to the eight warps of one block -- while this call uses a fixed size, so the two add the same terms in
            # different groupings and round the bf16 output differently by an ulp here and there: tolerance, not
            # bits; row by row for the reason given below) ...
            assert max(rel_err(got[s], o_stage[s]) for s in range(n)) <= TOL
            # ... and against the oracle's attention of the same bf16 queries over the same cache
            # (row by row: a sequence of 6 keys has outputs of the size of V itself, one of 1500 keys outputs thirty
            # times smaller, so one RMS over the whole tensor would measure the short rows by the long ones' scale)
            want = _oracle_attention(orc, case, dims, q.float().cpu().numpy(), pool_bits, kv_len)
            err = max(rel_err(got[s], want[s]) for s in range(n))
            print(f"no-alloc decode attention, head_dim {dims.head_dim}: max|err|/RMS(row) vs oracle = {err:.2e}")
            assert err <= TOL
            # a smaller SM budget changes nothing
            o_b = torch.empty_like(o_got)
            B.hs_op_decode_attention_noalloc(*args, o_b.data_ptr(), 7)
            torch.cuda.synchronize()
            assert torch.equal(o_b, o_got)
            kept.append((st, case, args, o_got, q))   # q stays alive: args holds its address
            st = None
        finally:
            if st is not None:
                st.close()
    try:
        # the two problems back to back on one stream, no synchronisation in between: the second call's metadata
        # and queue heads replace the first one's only after the first kernel has finished
        stream = torch.cuda.Stream(device=dev)
        outs = [torch.full_like(k[3], float("nan")) for k in kept]
        for k, o in zip(kept, outs):
            B.hs_op_decode_attention_noalloc(*k[2], o.data_ptr(), 148, stream.cuda_stream)
        stream.synchronize()
        assert B.hs_op_decode_attention_noalloc_status() == B.HS_OK
        for k, o in zip(kept, outs):
            assert torch.equal(o, k[3])
    finally:
        for k in kept:
            k[0].close()
