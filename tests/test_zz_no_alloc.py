"""hs_op_decode_attention_noalloc: the decode-attention variant for callers that cannot allocate device
memory (all HBM already given to the KV pool, or a component that only ever receives pointers).  Its
scratch is a fixed array inside the library, shared by every call, so the checks are: same result as
the regular path (the decode attention inside hs_stage_step, read back through the stage's "o" buffer),
on two different calls in a row -- the second one must not see anything the first one left behind --
and a clear refusal of problems larger than the fixed scratch.

Collected last on purpose: a run that stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2608_01785_b200 import binding as B
from paper_2608_01785_b200 import workloads as wl
from tests.helpers import make_case, rel_err

TOL = 2e-2


def test_sizes_beyond_the_fixed_scratch_are_refused():
    """Host-side checks come first, so this needs no GPU: nothing is launched for an oversized problem."""
    bt = np.zeros((1, 8), dtype=np.int32)
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
    del bt


def _decode_case(dims, ctx_len, seed):
    batch = wl.BatchSpec([1] * len(ctx_len), list(ctx_len))
    return make_case(dims, batch, seed=seed, kv_fill=True)


@pytest.mark.gpu
def test_noalloc_decode_attention_matches_the_stage_path_twice_in_a_row():
    from tests.gpu_helpers import make_stage, run_step
    dev = torch.device("cuda:0")
    problems = [
        (wl.StageDims(1, 512, 8, 2, 64, 1024), [700, 33, 255, 256, 1023, 5, 64, 300], 31),
        (wl.StageDims(1, 512, 8, 1, 128, 1024), [40, 1500, 511, 17], 32),   # other head size, fewer and longer
    ]
    for dims, ctx, seed in problems:
        case = _decode_case(dims, ctx, seed)
        st = make_stage(case, flags=B.HS_FLAG_BF16_ACTIVATIONS)   # the stage's o in bf16, as this call writes it
        try:
            run_step(st, case, 148)
            n = case.batch.n_seqs
            q = st.debug_tensor("q")[:n].contiguous()            # queries after RoPE, as the stage used them
            o_want = st.debug_tensor("o")[:n].float().cpu().numpy()
            o_got = torch.full((n, dims.q_dim), float("nan"), dtype=torch.bfloat16, device=dev)
            kv_len = [c + 1 for c in ctx]                          # the step cached the new token as well
            B.hs_op_decode_attention_noalloc(q.data_ptr(), st.kv_pool.data_ptr(), dims.n_layers, 0,
                                             case.cfg.num_pages, dims.n_q_heads, dims.n_kv_heads, dims.head_dim,
                                             kv_len, case.block_tables, o_got.data_ptr(), 148)
            torch.cuda.synchronize()
            got = o_got.float().cpu().numpy()
            assert np.all(np.isfinite(got))
            assert rel_err(got, o_want) <= TOL
            assert np.array_equal(got, o_want)                   # same kernels, same split: same bits
            # a smaller SM budget changes nothing
            o_b = torch.empty_like(o_got)
            B.hs_op_decode_attention_noalloc(q.data_ptr(), st.kv_pool.data_ptr(), dims.n_layers, 0,
                                             case.cfg.num_pages, dims.n_q_heads, dims.n_kv_heads, dims.head_dim,
                                             kv_len, case.block_tables, o_b.data_ptr(), 7)
            torch.cuda.synchronize()
            assert torch.equal(o_b, o_got)
        finally:
            st.close()
