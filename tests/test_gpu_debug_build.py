"""The bounds-checked debug library (libdash_attn_debug.so, -DDASH_DEBUG): kernels that index memory with values they
read from device memory (routed-chunk lists, counts) check them first; a bad value records DASH_ERR_CAPACITY in the
status word and the access is skipped -- nothing traps or faults.  The malformed lists below are only ever handed to
the debug library."""
import pytest
import torch

from paper_2605_18753_b200 import binding as B
from paper_2605_18753_b200 import synth
from tests.test_gpu_parity import _wl

pytestmark = pytest.mark.gpu
DEV = "cuda"
DASH_ERR_CAPACITY = -4


def _decode_setup(dtype):
    w = _wl(kind="decode", batch=2, seq=2048, h_q=8, h_kv=2, head_dim=128, block=64, dtype=dtype)
    inp = synth.make_decode_inputs(w, DEV, kv_len=[2048, 1000])
    q, Kc, Vc, lens = inp["Q"], inp["K"], inp["V"], inp["kv_len"]
    o = torch.empty_like(q)
    p = B.params_for_decode(q, Kc, Vc, o, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, Kc, kbar, kv_len=lens)
    ws = B.alloc_workspace(p)
    rt = B.alloc_routing(p)
    B.dash_attn_select(p, q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws, kv_len=lens)
    return w, p, q, Kc, Vc, lens, rt, ws


@pytest.mark.parametrize("dtype", ["bf16", "f32"])        # tensor-core kernel / CUDA-core kernel
def test_debug_library_matches_and_catches_malformed_lists(dtype):
    # valid routing from the production library
    w, p, q, Kc, Vc, lens, rt, ws = _decode_setup(dtype)
    want = torch.empty_like(q)
    B.dash_attn_attend_decode(p, q, Kc, Vc, lens, rt["count"], rt["blk_idx"], rt["blk_bias"], want, ws)
    assert B.dash_attn_last_status(ws) == 0
    assert int(rt["count"].min()) >= 1

    with B.use_debug_library():
        got = torch.full_like(q, float("nan"))
        B.dash_attn_attend_decode(p, q, Kc, Vc, lens, rt["count"], rt["blk_idx"], rt["blk_bias"], got, ws)
        assert B.dash_attn_last_status(ws) == 0
        # the checks change nothing on valid input (the CUDA-core kernels may contract their fp32 arithmetic differently
        # in the two builds: last-bit differences only)
        assert torch.allclose(got.float(), want.float(), rtol=0, atol=0 if dtype == "bf16" else 1e-6)

        # a chunk id far outside the cache
        bad_idx = rt["blk_idx"].clone()
        bad_idx[0] = 1 << 20
        B.dash_attn_attend_decode(p, q, Kc, Vc, lens, rt["count"], bad_idx, rt["blk_bias"], got, ws)
        assert B.dash_attn_last_status(ws) == DASH_ERR_CAPACITY
        B.dash_attn_reset_status(ws)

        # a negative chunk id
        bad_idx = rt["blk_idx"].clone()
        bad_idx[0] = -5
        B.dash_attn_attend_decode(p, q, Kc, Vc, lens, rt["count"], bad_idx, rt["blk_bias"], got, ws)
        assert B.dash_attn_last_status(ws) == DASH_ERR_CAPACITY
        B.dash_attn_reset_status(ws)

        # a count larger than the list can hold
        bad_count = rt["count"].clone()
        bad_count.view(-1)[1] = 1 << 24
        B.dash_attn_attend_decode(p, q, Kc, Vc, lens, bad_count, rt["blk_idx"], rt["blk_bias"], got, ws)
        assert B.dash_attn_last_status(ws) == DASH_ERR_CAPACITY
        B.dash_attn_reset_status(ws)

        # and the context is intact: the valid call still gives the right answer
        B.dash_attn_attend_decode(p, q, Kc, Vc, lens, rt["count"], rt["blk_idx"], rt["blk_bias"], got, ws)
        assert B.dash_attn_last_status(ws) == 0
        assert torch.allclose(got.float(), want.float(), rtol=0, atol=0 if dtype == "bf16" else 1e-6)
    # back on the production library
    assert B.LIB_PATH.endswith("libdash_attn.so")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_debug_library_catches_page_ids_outside_the_pool(dtype):
    from tests.test_gpu_paged import _scatter_into_pages
    w = _wl(kind="decode", batch=2, seq=2048, h_q=8, h_kv=2, head_dim=128, block=64, dtype=dtype)
    inp = synth.make_decode_inputs(w, DEV, kv_len=[2048, 1000])
    q, Kc, Vc, lens = inp["Q"], inp["K"], inp["V"], inp["kv_len"]
    Kpool, Vpool, table = _scatter_into_pages(Kc, Vc, 128, seed=5)
    o = torch.empty_like(q)
    pp = B.params_for_paged_decode(q, Kpool, Vpool, o, max_pages=table.shape[1], block=w.block, alpha=w.alpha,
                                   gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(pp)
    B.dash_attn_block_summaries_paged(pp, Kpool, table, kbar, kv_len=lens)     # production library, valid table
    ws = B.alloc_workspace(pp)
    want = torch.empty_like(q)
    B.dash_attn_fwd_decode_paged(pp, q, Kpool, Vpool, table, kbar, lens, want, ws)
    assert B.dash_attn_last_status(ws) == 0

    with B.use_debug_library():
        B.dash_attn_fwd_decode_paged(pp, q, Kpool, Vpool, table, kbar, lens, o, ws)
        assert B.dash_attn_last_status(ws) == 0
        assert torch.allclose(o.float(), want.float(), rtol=0, atol=0 if dtype == "bf16" else 1e-6)
        # Stage 2 is the only stage of this call that follows the page table (the summaries are given): every page of
        # sequence 0 is attended (its own chunk sits in the last one), so any bad entry of that row is met
        for bad in (Kpool.shape[0] + 7, -1):
            t2 = table.clone()
            t2[0, -1] = bad
            B.dash_attn_fwd_decode_paged(pp, q, Kpool, Vpool, t2, kbar, lens, o, ws)
            assert B.dash_attn_last_status(ws) == DASH_ERR_CAPACITY
            B.dash_attn_reset_status(ws)
        B.dash_attn_fwd_decode_paged(pp, q, Kpool, Vpool, table, kbar, lens, o, ws)
        assert B.dash_attn_last_status(ws) == 0
        assert torch.allclose(o.float(), want.float(), rtol=0, atol=0 if dtype == "bf16" else 1e-6)
