"""dash_attn_attend_decode_static: decode attention for callers that may not allocate device memory.

Such a caller (a serving loop with a frozen memory plan, a plugin whose host owns the allocator) cannot
give the library a workspace, so this entry point keeps the split-KV partials in a fixed array inside the
library.  The test calls it through the C ABI twice in a row and checks both results against
dash_attn_attend_decode (same routed lists, caller-provided workspace).  It lives in a file that pytest
collects last so that a run stopping at the first failure has already run everything else; it also
passes on its own in a fresh process.
"""
import ctypes

import pytest
import torch

from paper_2605_18753_b200 import binding as B
from paper_2605_18753_b200 import synth

pytestmark = pytest.mark.gpu


def _decode_problem(seed):
    w = synth.Workload("na", "decode", 3, 4096, 16, 4, 128, 64, 1.5, "bf16", "planted", n_planted=4, seed=seed)
    di = synth.make_decode_inputs(w, "cuda", kv_len=[4096, 3000, 65])
    q, Kc, Vc, lens = di["Q"], di["K"], di["V"], di["kv_len"]
    o = torch.empty_like(q)
    p = B.params_for_decode(q, Kc, Vc, o, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, Kc, kbar, kv_len=lens)
    ws = B.alloc_workspace(p)
    rt = B.alloc_routing(p)
    B.dash_attn_select(p, q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws, kv_len=lens)
    return p, q, Kc, Vc, lens, rt, ws


def test_static_scratch_decode_matches_workspace_decode_twice():
    for seed in (0, 1):                       # two different problems back to back: nothing may leak between calls
        p, q, Kc, Vc, lens, rt, ws = _decode_problem(seed)
        want = torch.full_like(q, float("nan"))
        B.dash_attn_attend_decode(p, q, Kc, Vc, lens, rt["count"], rt["blk_idx"], rt["blk_bias"], want, ws)
        assert B.dash_attn_last_status(ws) == 0
        for call in range(2):
            got = torch.full_like(q, float("nan"))
            B.dash_attn_attend_decode_static(p, q, Kc, Vc, lens, rt["count"], rt["blk_idx"], rt["blk_bias"], got)
            torch.cuda.synchronize()
            assert torch.isfinite(got.float()).all()
            err = (got.float() - want.float()).abs()
            assert err.max().item() <= 2e-2 and err.mean().item() <= 2e-3, (seed, call, err.max().item())


def test_static_scratch_rejects_problems_beyond_its_array():
    # 64 sequences x 128 query heads x 2 splits x 130 floats = 8.5 MiB > 4 MiB: refused before any launch
    p = B.make_params(batch=64, seq_q=1, seq_kv=4096, h_q=128, h_kv=8, head_dim=128, block=64, dtype=B.DASH_BF16,
                      alpha=1.5)
    rc = B.lib().dash_attn_attend_decode_static(ctypes.byref(p), 256, 256, 256, None, 256, 256, 256, 256, None)
    assert rc == -8 and "static" in B.strerror(rc)
