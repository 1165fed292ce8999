"""dash_attn_attend_decode_static: decode attention for callers that may not allocate device memory.

Such a caller (a serving loop with a frozen memory plan, a plugin whose host owns the allocator) cannot
give the library a workspace, so this entry point keeps the split-KV partials in a fixed array inside the
library.  The tests call it through the C ABI twice in a row and check both results against
dash_attn_attend_decode (same routed lists, caller-provided workspace) and against the float64 oracle, on
several shapes (bf16 and fp32, head_dim 128 and 64, group sizes 4 and 1, with and without kv_len), and check
that a call leaves the device's free memory and torch's allocator untouched.  The file is collected last so
that a run stopping at the first failure has already run everything else; it also passes on its own in a
fresh process.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import dash_oracle as orc
from paper_2605_18753_b200 import binding as B
from paper_2605_18753_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

SHAPES = {
    "bf16_d128_g4": dict(batch=3, seq=4096, h_q=16, h_kv=4, head_dim=128, block=64, dtype="bf16", kv_len=[4096, 3000, 65]),
    "f32_d64_g1": dict(batch=2, seq=1500, h_q=2, h_kv=2, head_dim=64, block=32, dtype="f32", kv_len=[1500, 700]),
    "bf16_d64_g4_full_cache": dict(batch=2, seq=2048, h_q=8, h_kv=2, head_dim=64, block=64, dtype="bf16", kv_len=None),
}


def _decode_problem(shape, seed):
    kw = dict(SHAPES[shape])
    kv_len = kw.pop("kv_len")
    w = synth.Workload("na", "decode", kw["batch"], kw["seq"], kw["h_q"], kw["h_kv"], kw["head_dim"], kw["block"], 1.5,
                       kw["dtype"], "planted", n_planted=4, seed=seed)
    di = synth.make_decode_inputs(w, "cuda", kv_len=kv_len)
    q, Kc, Vc = di["Q"], di["K"], di["V"]
    lens = di["kv_len"] if kv_len is not None else None      # None: the call gets kv_len = NULL (whole cache valid)
    o = torch.empty_like(q)
    p = B.params_for_decode(q, Kc, Vc, o, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, Kc, kbar, kv_len=lens)
    ws = B.alloc_workspace(p)
    rt = B.alloc_routing(p)
    B.dash_attn_select(p, q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws, kv_len=lens)
    return w, p, q, Kc, Vc, lens, di["kv_len"], rt, ws


@pytest.mark.parametrize("shape", sorted(SHAPES))
def test_static_scratch_decode_matches_workspace_decode_and_oracle_twice(shape):
    for seed in (0, 1):                       # two different problems back to back: nothing may leak between calls
        w, p, q, Kc, Vc, lens, lens_full, rt, ws = _decode_problem(shape, seed)
        want = torch.full_like(q, float("nan"))
        B.dash_attn_attend_decode(p, q, Kc, Vc, lens, rt["count"], rt["blk_idx"], rt["blk_bias"], want, ws)
        assert B.dash_attn_last_status(ws) == 0
        # the oracle's Stage 2 on the lists the GPU routed (Stage 1 has its own parity tests)
        Qn, Kn, Vn = H.to_np64(q), H.to_np64(Kc), H.to_np64(Vc)
        cnt = rt["count"].cpu().numpy()
        idx = rt["blk_idx"].cpu().numpy()
        bias = rt["blk_bias"].cpu().numpy().astype(np.float64)
        g_q = w.h_q // w.h_kv
        ref = np.zeros((w.batch, w.h_q, w.head_dim))
        for b in range(w.batch):
            L = int(lens_full[b])
            for r in range(w.h_kv):
                off = B.dash_attn_list_offset(p, b, r, 0)
                c = int(cnt[b, r, 0])
                ref[b, r * g_q:(r + 1) * g_q] = orc.attend_row(Qn[b, r * g_q:(r + 1) * g_q], Kn[b, :L, r], Vn[b, :L, r],
                                                               w.block, idx[off:off + c], bias[off:off + c],
                                                               ((L - 1) // w.block) * w.block, L)
        mx, mean = H.tol_for(q.dtype)
        for call in range(2):
            got = torch.full_like(q, float("nan"))
            B.dash_attn_attend_decode_static(p, q, Kc, Vc, lens, rt["count"], rt["blk_idx"], rt["blk_bias"], got)
            torch.cuda.synchronize()
            assert torch.isfinite(got.float()).all()
            err = (got.float() - want.float()).abs()
            assert err.max().item() <= mx and err.mean().item() <= mean, (shape, seed, call, err.max().item())
            H.check_outputs(got.float().cpu().double().numpy(), ref, q.dtype, f"static decode vs oracle {shape}")


def test_static_scratch_call_allocates_nothing():
    """After the first call on the device (which looks up the array's address), a call must leave the device's
    free memory and torch's caching allocator exactly as they were."""
    w, p, q, Kc, Vc, lens, _, rt, ws = _decode_problem("bf16_d128_g4", 2)
    got = torch.empty_like(q)
    B.dash_attn_attend_decode_static(p, q, Kc, Vc, lens, rt["count"], rt["blk_idx"], rt["blk_bias"], got)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        B.dash_attn_attend_decode_static(p, q, Kc, Vc, lens, rt["count"], rt["blk_idx"], rt["blk_bias"], got)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0


def test_static_scratch_rejects_problems_beyond_its_array():
    # 64 sequences x 128 query heads x >= 1 split x 130 floats >= 4.06 MiB > 4 MiB: refused before any launch
    p = B.make_params(batch=64, seq_q=1, seq_kv=4096, h_q=128, h_kv=8, head_dim=128, block=64, dtype=B.DASH_BF16,
                      alpha=1.5)
    rc = B.lib().dash_attn_attend_decode_static(ctypes.byref(p), 256, 256, 256, None, 256, 256, 256, 256, None)
    assert rc == -8 and "static" in B.strerror(rc)
    # the documented safe bound: batch * h_q * 32 * (head_dim + 2) * 4 bytes <= 4 MiB is never refused for its size
    p = B.make_params(batch=4, seq_q=1, seq_kv=4096, h_q=32, h_kv=8, head_dim=128, block=64, dtype=B.DASH_BF16, alpha=1.5)
    assert 4 * 32 * 32 * 130 * 4 <= 4 << 20
    rc = B.lib().dash_attn_attend_decode_static(ctypes.byref(p), None, 256, 256, None, 256, 256, 256, 256, None)
    assert rc == -1          # a null Q is an argument error, not TOO_LARGE: the size check passed
