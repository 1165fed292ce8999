"""Paged KV cache: the decode step over a block-table cache must give what the contiguous cache gives (the same
tiles are fetched, only from other addresses) and match the float64 oracle run on the logically contiguous cache."""
import numpy as np
import pytest
import torch

from oracle import dash_oracle as orc
from paper_2605_18753_b200 import binding as B
from paper_2605_18753_b200 import synth
from tests import helpers as H
from tests.test_gpu_parity import _wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _scatter_into_pages(Kc, Vc, page_size, seed, spare=3):
    """Cuts the contiguous caches [b, cap, h, d] into pages and scatters them over a pool in a seeded random order
    (plus a few unused pages filled with NaN).  Returns (Kpool, Vpool, page_table [b, max_pages] int32)."""
    b, cap, h, d = Kc.shape
    assert cap % page_size == 0
    max_pages = cap // page_size
    n_pages = b * max_pages + spare
    perm = torch.randperm(n_pages, generator=torch.Generator().manual_seed(seed))[: b * max_pages]
    table = perm.view(b, max_pages).to(torch.int32)
    Kpool = torch.full((n_pages, page_size, h, d), float("nan"), dtype=Kc.dtype, device=Kc.device)
    Vpool = torch.full_like(Kpool, float("nan"))
    idx = table.to(Kc.device).long().view(-1)
    Kpool[idx] = Kc.view(b * max_pages, page_size, h, d)
    Vpool[idx] = Vc.view(b * max_pages, page_size, h, d)
    return Kpool, Vpool, table.to(Kc.device)


@pytest.mark.parametrize("kw,kv_len,page_size", [
    (dict(kind="decode", batch=3, seq=2048, h_q=8, h_kv=2, head_dim=128, block=64), [2048, 1, 777], 64),
    (dict(kind="decode", batch=2, seq=4096, h_q=16, h_kv=2, head_dim=128, block=64), [4096, 2500], 256),
    (dict(kind="decode", batch=2, seq=3072, h_q=4, h_kv=2, head_dim=128, block=128, alpha=2.0), [3000, 2050], 128),
    (dict(kind="decode", batch=2, seq=2560, h_q=8, h_kv=2, head_dim=128, block=32), [2500, 33], 128),      # packed chunks
    (dict(kind="decode", batch=2, seq=2048, h_q=16, h_kv=2, head_dim=64, block=16, alpha=1.25, gamma=2.0), [1800, 1001], 64),
    (dict(kind="decode", batch=2, seq=1536, h_q=2, h_kv=2, head_dim=128, block=64, dtype="f32"), [1500, 65], 192),   # CUDA-core path
])
def test_paged_decode_equals_contiguous_decode_and_oracle(kw, kv_len, page_size):
    w = _wl(**kw)
    inp = synth.make_decode_inputs(w, DEV, kv_len=kv_len)
    Q, Kc, Vc, lens = inp["Q"], inp["K"], inp["V"], inp["kv_len"]
    # contiguous reference run
    O_ref = torch.full_like(Q, float("nan"))
    pc = B.params_for_decode(Q, Kc, Vc, O_ref, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar_c = B.alloc_kbar(pc)
    kbar_c.fill_(float("nan"))
    B.dash_attn_block_summaries(pc, Kc, kbar_c, kv_len=lens)
    wsc = B.alloc_workspace(pc)
    B.dash_attn_fwd_decode(pc, Q, Kc, Vc, kbar_c, lens, O_ref, wsc)
    assert B.dash_attn_last_status(wsc) == 0

    Kpool, Vpool, table = _scatter_into_pages(Kc, Vc, page_size, seed=w.seq + page_size)
    O = torch.full_like(Q, float("nan"))
    pp = B.params_for_paged_decode(Q, Kpool, Vpool, O, max_pages=table.shape[1], block=w.block, alpha=w.alpha,
                                   gamma=w.gamma, sigma=w.sigma)
    assert pp.seq_kv == w.seq
    kbar = B.alloc_kbar(pp)
    kbar.fill_(float("nan"))
    B.dash_attn_block_summaries_paged(pp, Kpool, table, kbar, kv_len=lens)
    # summaries of complete chunks are bit-identical (same arithmetic, other addresses); the rest stays untouched
    both = ~torch.isnan(kbar_c)
    assert torch.equal(torch.isnan(kbar), torch.isnan(kbar_c)) and torch.equal(kbar[both], kbar_c[both])
    ws = B.alloc_workspace(pp)
    B.dash_attn_fwd_decode_paged(pp, Q, Kpool, Vpool, table, kbar, lens, O, ws)
    assert B.dash_attn_last_status(ws) == 0
    assert torch.isfinite(O.float()).all()
    assert torch.equal(O, O_ref)

    # and against the oracle on the contiguous cache (rows whose routing holds a borderline chunk are left out)
    ora = orc.forward_decode(H.to_np64(Q), H.to_np64(Kc), H.to_np64(Vc), lens.cpu().numpy(), B=w.block, alpha=w.alpha,
                             gamma=w.gamma, sigma=w.sigma)
    g_q = w.h_q // w.h_kv
    clean = np.ones((w.batch, w.h_kv), dtype=bool)
    for (b, r), ro in ora["routing"].items():
        clean[b, r] = not (ro.n_cand and (np.abs(ro.margin) <= H.BORDERLINE).any())
    sel = np.repeat(clean, g_q, axis=1)
    assert sel.any()
    H.check_outputs(O.float().cpu().double().numpy()[sel], ora["O"][sel], Q.dtype, "paged decode")


def test_paged_entry_points_reject_bad_page_geometry():
    w = _wl(kind="decode", batch=1, seq=1024, h_q=4, h_kv=2, head_dim=128, block=64)
    inp = synth.make_decode_inputs(w, DEV)
    Q, Kc, Vc = inp["Q"], inp["K"], inp["V"]
    O = torch.empty_like(Q)
    Kpool, Vpool, table = _scatter_into_pages(Kc, Vc, 128, seed=1)
    pp = B.params_for_paged_decode(Q, Kpool, Vpool, O, max_pages=table.shape[1], block=64, alpha=1.5)
    kbar = B.alloc_kbar(pp)
    ws = B.alloc_workspace(pp)
    L = B.lib()
    import ctypes
    args = lambda ps, mp: (ctypes.byref(pp), Q.data_ptr(), Kpool.data_ptr(), Vpool.data_ptr(), table.data_ptr(), ps, mp,
                           Kpool.shape[0], kbar.data_ptr(), None, O.data_ptr(), ws.data_ptr(), ws.numel(), None)
    assert L.dash_attn_fwd_decode_paged(*args(96, 8)) == -1          # not a multiple of 64
    assert L.dash_attn_fwd_decode_paged(*args(128, 7)) == -1         # max_pages * page_size != seq_kv
    assert L.dash_attn_fwd_decode_paged(*args(128, 8)) == 0
    torch.cuda.synchronize()
