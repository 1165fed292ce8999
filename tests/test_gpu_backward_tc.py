"""GPU parity of the tensor-core Stage-2 backward (dash_attn_bwd_attend_prefill_tc): against the float64 backward oracle
on the oracle's own routing lists (every row, every gradient), and against the CUDA-core backward kernel on a larger
case with the library's routing.  P and dS enter the dK / dV products rounded to bf16 and dQ is stored as bf16: those
three carry the bf16 tolerance (1e-2 of the largest reference value).  dbias is formed from fp32 values (delta comes
from a statistics pass that feeds P to its P V product as two bf16 terms), because the routing's backward amplifies its
error: 2e-3 of the largest reference value, and the whole chain through the routing is checked as well."""
import numpy as np
import pytest
import torch

from oracle import dash_oracle_bwd as bwd
from paper_2605_18753_b200 import binding as B
from paper_2605_18753_b200 import synth
from tests import helpers as H
from tests.test_gpu_backward import _close, whole_chain_case
from tests.test_gpu_parity import _wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _run_tc(p, Q, K, V, dO, mask, bias, w):
    dQ = torch.full_like(Q, float("nan"))
    dK = torch.full((w.batch, w.seq, w.h_kv, w.head_dim), float("nan"), device=DEV)
    dV = torch.full_like(dK, float("nan"))
    dbias = torch.full((max(B.dash_attn_list_capacity(p), 1),), float("nan"), device=DEV)
    bws = B.alloc_bwd_workspace(p)
    B.dash_attn_bwd_attend_prefill_tc(p, Q, K, V, dO, mask, bias, dQ, dK, dV, dbias, bws)
    torch.cuda.synchronize()
    assert B.dash_attn_last_status(bws) == 0
    return dQ, dK, dV, dbias


@pytest.mark.parametrize("kw,L", [
    (dict(seq=400, h_q=8, h_kv=2, head_dim=128, block=64, sigma=1.0), 0),
    (dict(seq=700, h_q=4, h_kv=2, head_dim=128, block=128, seed=21, sigma=2.0), 0),      # two steps per chunk, g_q = 2
    (dict(seq=333, h_q=8, h_kv=1, head_dim=128, block=64, alpha=2.0, seed=22), 0),        # g_q = 8, ragged length
    (dict(seq=520, h_q=8, h_kv=2, head_dim=128, block=64, batch=2, seed=23, gamma=2.0), 0),
    (dict(seq=420, h_q=4, h_kv=1, head_dim=128, block=64, seed=24), 1),                   # local window
    (dict(seq=300, h_q=16, h_kv=1, head_dim=128, block=64, seed=27, gamma=2.0), 0),       # g_q = 16: tiles of 8 tokens
    (dict(seq=64, h_q=4, h_kv=2, head_dim=128, block=64, seed=25), 0),                    # one chunk: nothing routed
    (dict(seq=5, h_q=4, h_kv=2, head_dim=128, block=64, seed=26), 0),
])
def test_tensor_core_stage2_backward_matches_oracle(kw, L):
    w = _wl(**kw)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    dO = torch.randn(Q.shape, device=DEV, generator=torch.Generator(DEV).manual_seed(w.seed + 190)).to(Q.dtype)
    p = B.params_for_prefill(Q, K, V, dO, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, local_blocks=L)
    Qn, Kn, Vn, Gn = (H.to_np64(t) for t in (Q, K, V, dO))
    kwo = dict(B=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, local_blocks=L)
    ora = H.oracle_prefill_rows(Q, K, V, rows=range(w.seq), **kwo)
    mask, count, idx, bias = H.routing_to_abi(ora, p, B.dash_attn_list_offset)
    ref = bwd.backward_prefill(Qn, Kn, Vn, Gn, through_routing=False, **kwo)
    dQ, dK, dV, dbias = _run_tc(p, Q, K, V, dO, mask, bias, w)
    _close(dQ.float().cpu().double().numpy(), ref["dQ"], 1e-2, "dQ")
    _close(dK.cpu().double().numpy(), ref["dK"], 1e-2, "dK")
    _close(dV.cpu().double().numpy(), ref["dV"], 1e-2, "dV")
    db = dbias.cpu().double().numpy()
    n_entries = 0
    scale = max([1.0] + [float(np.abs(v).max()) for v in ref["dbias"].values() if v.size])
    for (b, r, i), want in ref["dbias"].items():
        off = B.dash_attn_list_offset(p, b, r, i)
        if want.size:
            err = float(np.abs(db[off:off + want.size] - want).max())
            assert err <= 2e-3 * scale, f"dbias row {(b, r, i)}: {err:.3e} vs scale {scale:.3g}"
            n_entries += want.size
    if w.seq > 4 * w.block:
        assert n_entries > 0
    # entries outside every row's count are zeroed as well
    if B.dash_attn_list_capacity(p) > 0:
        assert np.isfinite(db).all()


def test_tensor_core_backward_equals_cuda_core_backward_on_library_routing():
    w = _wl(seq=2048 + 37, h_q=8, h_kv=2, head_dim=128, block=64, seed=31, batch=2)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    dO = torch.randn(Q.shape, device=DEV, generator=torch.Generator(DEV).manual_seed(131)).to(Q.dtype)
    p = B.params_for_prefill(Q, K, V, dO, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, K, kbar)
    ws = B.alloc_workspace(p)
    rt = B.alloc_routing(p)
    B.dash_attn_select(p, Q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws)
    assert int(rt["count"].max()) > 0
    dQ0 = torch.empty_like(Q)
    dK0 = torch.empty(w.batch, w.seq, w.h_kv, w.head_dim, device=DEV)
    dV0 = torch.empty_like(dK0)
    db0 = torch.empty_like(rt["blk_bias"])
    B.dash_attn_bwd_attend_prefill(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], dQ0, dK0, dV0, db0)
    dQ, dK, dV, db = _run_tc(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], w)
    for got, want, what, rel in ((dQ, dQ0, "dQ", 1e-2), (dK, dK0, "dK", 1e-2), (dV, dV0, "dV", 1e-2), (db, db0, "dbias", 1e-2)):
        _close(got.float().cpu().double().numpy(), want.float().cpu().double().numpy(), rel, what)
    # a second run gives the same bits (no atomics on dQ, dK, dV; one or two commutative adds per dbias entry)
    dQ2, dK2, dV2, db2 = _run_tc(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], w)
    assert torch.equal(dQ, dQ2) and torch.equal(dK, dK2) and torch.equal(dV, dV2) and torch.equal(db, db2)


def test_tensor_core_backward_refuses_other_shapes():
    w = _wl(seq=300, h_q=4, h_kv=2, head_dim=128, block=32, seed=5)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    p = B.params_for_prefill(Q, K, V, Q, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    rt = B.alloc_routing(p)
    bws = B.alloc_bwd_workspace(p)
    dK = torch.empty(w.batch, w.seq, w.h_kv, w.head_dim, device=DEV)
    with pytest.raises(B.DashError) as ei:
        B.dash_attn_bwd_attend_prefill_tc(p, Q, K, V, Q, rt["mask"], rt["blk_bias"], torch.empty_like(Q), dK,
                                          torch.empty_like(dK), torch.empty_like(rt["blk_bias"]), bws)
    assert ei.value.code == -2


@pytest.mark.parametrize("kw,qbar_mode,L", [
    (dict(seq=400, h_q=8, h_kv=2, head_dim=128, block=64, sigma=1.0, seed=14), "none", 0),
    (dict(seq=520, h_q=4, h_kv=2, head_dim=128, block=128, sigma=2.0, seed=41), "head", 0),
    (dict(seq=420, h_q=4, h_kv=2, head_dim=128, block=64, seed=17, sigma=2.0), "chunk", 1),
])
def test_whole_backward_chain_with_tensor_core_stage2(kw, qbar_mode, L):
    """The whole gradient chain of the method with Stage 2 on tensor cores (its dbias feeds the routing backward)."""
    whole_chain_case(kw, qbar_mode, L, tensor_cores=True)


def test_tensor_core_backward_gives_up_cleanly_when_a_wait_runs_out():
    """The statistics pass is the forward kernel: with the test hooks its first K tile never arrives and its waits give
    up after 2e5 cycles.  The status word of the backward scratch then holds DASH_ERR_TIMEOUT, the kernels behind it
    (launched on the same status word) retire at their first wait, nothing hangs or faults, and after a reset the same
    scratch serves a correct backward pass."""
    import time
    w = _wl(seq=900, h_q=8, h_kv=2, head_dim=128, block=64, seed=33)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    dO = torch.randn(Q.shape, device=DEV, generator=torch.Generator(DEV).manual_seed(133)).to(Q.dtype)
    p = B.params_for_prefill(Q, K, V, dO, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, K, kbar)
    ws = B.alloc_workspace(p)
    rt = B.alloc_routing(p)
    B.dash_attn_select(p, Q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws)
    bws = B.alloc_bwd_workspace(p)
    outs = lambda: (torch.full_like(Q, float("nan")), torch.empty(w.batch, w.seq, w.h_kv, w.head_dim, device=DEV),
                    torch.empty(w.batch, w.seq, w.h_kv, w.head_dim, device=DEV), torch.empty_like(rt["blk_bias"]))
    good = outs()
    B.dash_attn_bwd_attend_prefill_tc(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], *good, bws)
    assert B.dash_attn_last_status(bws) == 0
    try:
        B.dash_attn_test_hooks(wait_limit_cycles=200_000, skip_own_k_load=1)
        t0 = time.time()
        B.dash_attn_bwd_attend_prefill_tc(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], *outs(), bws)
        assert B.dash_attn_last_status(bws) == -7          # DASH_ERR_TIMEOUT
        assert time.time() - t0 < 5.0
    finally:
        B.dash_attn_test_hooks()
    torch.cuda.synchronize()
    B.dash_attn_reset_status(bws)
    again = outs()
    B.dash_attn_bwd_attend_prefill_tc(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], *again, bws)
    assert B.dash_attn_last_status(bws) == 0
    for g, a_ in zip(good, again):
        assert torch.equal(g, a_)


def test_tensor_core_backward_on_random_shapes_against_the_cuda_core_kernel():
    """Seeded random shapes inside the tensor-core path's domain (lengths that end inside a tile or a chunk, every group
    size, both chunk sizes, windows, batches), library routing, CUDA-core kernel as the reference (itself checked
    against the oracle above and in test_gpu_backward.py)."""
    rng = np.random.default_rng(20261125)
    for draw in range(14):
        g_q = int(rng.choice([2, 4, 8, 16]))
        h_kv = int(rng.choice([1, 2, 3]))
        kw = dict(seq=int(rng.integers(65, 1400)), h_q=g_q * h_kv, h_kv=h_kv, head_dim=128, block=int(rng.choice([64, 128])),
                  batch=int(rng.choice([1, 2])), alpha=float(rng.choice([1.25, 1.5, 2.0])), gamma=float(rng.choice([1.0, 2.0, 4.0])),
                  sigma=float(rng.choice([1.0, 10.0])), seed=100 + draw)
        L = int(rng.choice([0, 0, 1]))
        w = _wl(**kw)
        inp = synth.make_prefill_inputs(w, DEV)
        Q, K, V = inp["Q"], inp["K"], inp["V"]
        dO = torch.randn(Q.shape, device=DEV, generator=torch.Generator(DEV).manual_seed(500 + draw)).to(Q.dtype)
        p = B.params_for_prefill(Q, K, V, dO, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, local_blocks=L)
        kbar = B.alloc_kbar(p)
        B.dash_attn_block_summaries(p, K, kbar)
        ws = B.alloc_workspace(p)
        rt = B.alloc_routing(p)
        B.dash_attn_select(p, Q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws)
        assert B.dash_attn_last_status(ws) == 0
        dQ0 = torch.empty_like(Q)
        dK0 = torch.empty(w.batch, w.seq, w.h_kv, w.head_dim, device=DEV)
        dV0 = torch.empty_like(dK0)
        db0 = torch.empty_like(rt["blk_bias"])
        B.dash_attn_bwd_attend_prefill(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], dQ0, dK0, dV0, db0)
        dQ, dK, dV, db = _run_tc(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], w)
        what = f"draw {draw} {kw} L={L}"
        for got, want, name, rel in ((dQ, dQ0, "dQ", 1e-2), (dK, dK0, "dK", 1e-2), (dV, dV0, "dV", 1e-2), (db, db0, "dbias", 3e-3)):
            if want.numel():
                _close(got.float().cpu().double().numpy(), want.float().cpu().double().numpy(), rel, f"{name} ({what})")


def test_tensor_core_backward_at_the_full_8k_workload():
    """The workload bench.py times (prefill_8k, library routing): dQ rows and dbias entries of sampled rows against the
    float64 oracle's row-wise Stage-2 backward on the GPU's own lists, and all four gradients against the CUDA-core
    kernel."""
    w = synth.workload("prefill_8k")
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    dO = torch.randn(Q.shape, device=DEV, generator=torch.Generator(DEV).manual_seed(777)).to(Q.dtype)
    p = B.params_for_prefill(Q, K, V, dO, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, K, kbar)
    ws = B.alloc_workspace(p)
    rt = B.alloc_routing(p)
    B.dash_attn_select(p, Q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws)
    dQ, dK, dV, db = _run_tc(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], w)
    dQ0 = torch.empty_like(Q)
    dK0 = torch.empty(w.batch, w.seq, w.h_kv, w.head_dim, device=DEV)
    dV0 = torch.empty_like(dK0)
    db0 = torch.empty_like(rt["blk_bias"])
    B.dash_attn_bwd_attend_prefill(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], dQ0, dK0, dV0, db0)
    for got, want, name, rel in ((dQ, dQ0, "dQ", 1e-2), (dK, dK0, "dK", 1e-2), (dV, dV0, "dV", 1e-2), (db, db0, "dbias", 3e-3)):
        _close(got.float().cpu().double().numpy(), want.float().cpu().double().numpy(), rel, f"{name} vs the CUDA-core kernel")
    # sampled rows against the oracle
    Qn, Kn, Vn, Gn = (H.to_np64(t) for t in (Q, K, V, dO))
    cnt = rt["count"].cpu().numpy(); idx = rt["blk_idx"].cpu().numpy(); bias = rt["blk_bias"].cpu().numpy().astype(np.float64)
    dbn = db.cpu().double().numpy()
    dQn = dQ.float().cpu().double().numpy()
    g_q = w.h_q // w.h_kv
    rng = np.random.default_rng(5)
    scale_q = float(np.abs(dQn).max())
    for _ in range(48):
        r = int(rng.integers(0, w.h_kv)); i = int(rng.integers(0, w.seq))
        off = B.dash_attn_list_offset(p, 0, r, i)
        c = int(cnt[0, r, i])
        dq, tok, dk, dv, dbr = bwd.attend_row_vjp(Qn[0, i, r * g_q:(r + 1) * g_q], Kn[0, :, r], Vn[0, :, r], w.block,
                                                  idx[off:off + c], bias[off:off + c], (i // w.block) * w.block, i + 1,
                                                  Gn[0, i, r * g_q:(r + 1) * g_q])
        err = float(np.abs(dQn[0, i, r * g_q:(r + 1) * g_q] - dq).max())
        assert err <= 1e-2 * max(1.0, scale_q), f"dQ row {(r, i)}: {err:.3e}"
        if c:
            errb = float(np.abs(dbn[off:off + c] - dbr).max())
            assert errb <= 2e-3 * max(1.0, float(np.abs(dbr).max())), f"dbias row {(r, i)}: {errb:.3e}"
