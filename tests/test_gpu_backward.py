"""GPU parity of the Stage-2 backward kernel (dash_attn_bwd_attend_prefill) against the float64 backward oracle with
the routing held fixed, on the oracle's own routing lists: dQ, dK, dV and the gradient with respect to every bias entry."""
import numpy as np
import pytest
import torch

from oracle import dash_oracle as orc
from oracle import dash_oracle_bwd as bwd
from paper_2605_18753_b200 import binding as B
from paper_2605_18753_b200 import synth
from tests import helpers as H
from tests.test_gpu_parity import _wl

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _close(got, want, rel, what):
    scale = max(1.0, float(np.abs(want).max()))
    err = float(np.abs(got - want).max())
    assert np.isfinite(got).all(), what
    assert err <= rel * scale, f"{what}: max-abs {err:.3e} > {rel} * {scale:.3g}"
    return err


@pytest.mark.parametrize("kw,L", [
    (dict(seq=300, dtype="f32", gamma=3.0), 0),
    (dict(seq=400, h_q=8, h_kv=2, head_dim=128, block=64, sigma=1.0), 0),
    (dict(seq=333, h_q=4, h_kv=4, head_dim=128, block=32, alpha=2.0), 0),
    (dict(seq=500, h_q=8, h_kv=1, head_dim=64, block=16, gamma=2.0, alpha=1.25), 0),
    (dict(seq=17), 0), (dict(seq=5), 0),
    (dict(seq=420, h_q=4, h_kv=2, head_dim=128, block=64, seed=3), 1),          # local window
    (dict(seq=260, h_q=4, h_kv=2, head_dim=64, block=32, batch=2, seed=4), 0),
])
def test_stage2_backward_matches_oracle(kw, L):
    w = _wl(**kw)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    dO = (torch.randn(Q.shape, device=DEV, generator=torch.Generator(DEV).manual_seed(w.seed + 90)).to(Q.dtype))
    p = B.params_for_prefill(Q, K, V, dO, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, local_blocks=L)
    Qn, Kn, Vn, Gn = (H.to_np64(t) for t in (Q, K, V, dO))
    kwo = dict(B=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, local_blocks=L)
    ora = H.oracle_prefill_rows(Q, K, V, rows=range(w.seq), **kwo)
    mask, count, idx, bias = H.routing_to_abi(ora, p, B.dash_attn_list_offset)
    ref = bwd.backward_prefill(Qn, Kn, Vn, Gn, through_routing=False, **kwo)

    dQ = torch.full_like(Q, float("nan"))
    dK = torch.full((w.batch, w.seq, w.h_kv, w.head_dim), float("nan"), device=DEV)
    dV = torch.full_like(dK, float("nan"))
    dbias = torch.full((max(B.dash_attn_list_capacity(p), 1),), float("nan"), device=DEV)
    B.dash_attn_bwd_attend_prefill(p, Q, K, V, dO, mask, bias, dQ, dK, dV, dbias)
    torch.cuda.synchronize()
    fp32 = Q.dtype == torch.float32
    _close(dQ.float().cpu().double().numpy(), ref["dQ"], 2e-4 if fp32 else 1e-2, "dQ")
    _close(dK.cpu().double().numpy(), ref["dK"], 2e-4, "dK")
    _close(dV.cpu().double().numpy(), ref["dV"], 2e-4, "dV")
    db = dbias.cpu().double().numpy()
    n_entries = 0
    for (b, r, i), want in ref["dbias"].items():
        off = B.dash_attn_list_offset(p, b, r, i)
        if want.size:
            _close(db[off:off + want.size], want, 2e-4, f"dbias row {(b, r, i)}")
            n_entries += want.size
    if w.seq > 4 * w.block:
        assert n_entries > 0


def test_stage2_backward_on_the_library_routing():
    """The same comparison on the lists the library's own Stage 1 produced (mask, count, chunk ids and fp32 biases read
    back from the device), row by row through the oracle's Stage-2 backward."""
    w = _wl(seq=700, h_q=8, h_kv=2, head_dim=128, block=64, seed=8)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    dO = torch.randn(Q.shape, device=DEV, generator=torch.Generator(DEV).manual_seed(98)).to(Q.dtype)
    p = B.params_for_prefill(Q, K, V, dO, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, K, kbar)
    ws = B.alloc_workspace(p)
    rt = B.alloc_routing(p)
    B.dash_attn_select(p, Q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws)
    dQ = torch.empty_like(Q)
    dK = torch.empty(w.batch, w.seq, w.h_kv, w.head_dim, device=DEV)
    dV = torch.empty_like(dK)
    dbias = torch.empty_like(rt["blk_bias"])
    B.dash_attn_bwd_attend_prefill(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], dQ, dK, dV, dbias)
    torch.cuda.synchronize()
    # oracle Stage-2 backward on the GPU's lists, row by row
    Qn, Kn, Vn, Gn = (H.to_np64(t) for t in (Q, K, V, dO))
    cnt = rt["count"].cpu().numpy(); idx = rt["blk_idx"].cpu().numpy(); bias = rt["blk_bias"].cpu().numpy().astype(np.float64)
    db = dbias.cpu().double().numpy()
    g_q = w.h_q // w.h_kv
    dQ_ref = np.zeros_like(Qn); dK_ref = np.zeros_like(Kn); dV_ref = np.zeros_like(Vn)
    for r in range(w.h_kv):
        for i in range(w.seq):
            off = B.dash_attn_list_offset(p, 0, r, i)
            c = int(cnt[0, r, i])
            dq, tok, dk, dv, dbr = bwd.attend_row_vjp(Qn[0, i, r * g_q:(r + 1) * g_q], Kn[0, :, r], Vn[0, :, r], w.block,
                                                      idx[off:off + c], bias[off:off + c], (i // w.block) * w.block, i + 1,
                                                      Gn[0, i, r * g_q:(r + 1) * g_q])
            dQ_ref[0, i, r * g_q:(r + 1) * g_q] = dq
            np.add.at(dK_ref[0, :, r], tok, dk)
            np.add.at(dV_ref[0, :, r], tok, dv)
            if c:
                _close(db[off:off + c], dbr, 2e-4, f"dbias row {(r, i)}")
    _close(dQ.float().cpu().double().numpy(), dQ_ref, 1e-2, "dQ")
    _close(dK.cpu().double().numpy(), dK_ref, 2e-4, "dK")
    _close(dV.cpu().double().numpy(), dV_ref, 2e-4, "dV")


@pytest.mark.parametrize("kw,qbar_mode,L", [
    (dict(seq=300, dtype="f32", gamma=3.0, sigma=2.0), "none", 0),
    (dict(seq=400, h_q=8, h_kv=2, head_dim=128, block=64, sigma=1.0, seed=14), "none", 0),
    (dict(seq=333, h_q=4, h_kv=4, head_dim=128, block=32, alpha=2.0, sigma=2.0, seed=15), "head", 0),
    (dict(seq=420, h_q=8, h_kv=1, head_dim=64, block=16, gamma=2.0, alpha=1.25, sigma=4.0, seed=16), "chunk", 0),
    (dict(seq=420, h_q=4, h_kv=2, head_dim=128, block=64, seed=17, sigma=2.0), "none", 1),      # local window
    (dict(seq=260, h_q=4, h_kv=2, head_dim=64, block=32, batch=2, seed=18, dtype="f32", sigma=1.0), "head", 0),
])
def test_whole_backward_chain_matches_oracle(kw, qbar_mode, L):
    """Stage 2, Stage 1 and Stage 0 backward kernels chained (dbias -> dQ through the routing and dKbar -> dK, dqbar)
    against the whole-method gradient of the float64 oracle, on the oracle's routing (mask, lists and thresholds)."""
    whole_chain_case(kw, qbar_mode, L, tensor_cores=False)


def whole_chain_case(kw, qbar_mode, L, tensor_cores):
    """tensor_cores: Stage 2 through dash_attn_bwd_attend_prefill_tc (bf16 tolerance on everything downstream of it)."""
    w = _wl(**kw)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    dO = torch.randn(Q.shape, device=DEV, generator=torch.Generator(DEV).manual_seed(w.seed + 91)).to(Q.dtype)
    p = B.params_for_prefill(Q, K, V, dO, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, local_blocks=L)
    T_s = w.seq // w.block
    qbar, stride = None, 0
    if qbar_mode == "head":
        qbar = torch.randn(w.h_kv, w.head_dim, device=DEV, generator=torch.Generator(DEV).manual_seed(w.seed + 52))
    elif qbar_mode == "chunk":
        qbar = torch.randn(T_s, w.h_kv, w.head_dim, device=DEV, generator=torch.Generator(DEV).manual_seed(w.seed + 53))
        stride = w.h_kv * w.head_dim
    qb64 = None if qbar is None else H.to_np64(qbar)
    Qn, Kn, Vn, Gn = (H.to_np64(t) for t in (Q, K, V, dO))
    kwo = dict(B=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, local_blocks=L)
    ora = H.oracle_prefill_rows(Q, K, V, rows=range(w.seq), qbar=qb64, **kwo)
    mask, count, idx, bias = H.routing_to_abi(ora, p, B.dash_attn_list_offset)
    g_q = w.h_q // w.h_kv
    tau = np.zeros((w.batch, w.h_q, w.seq), dtype=np.float32)
    for (b, r, i), (rt, _) in ora.items():
        if rt.n_cand:
            tau[b, r * g_q:(r + 1) * g_q, i] = rt.tau
    tau = torch.from_numpy(tau).to(DEV)
    ref = bwd.backward_prefill(Qn, Kn, Vn, Gn, qbar=qb64, through_routing=True, **kwo)
    # margins close to zero make the routing gradient arbitrarily large (d log w / d w = 1 / w): such inputs are a
    # property of the method, not of an implementation; the seeds above keep the smallest routed weight reasonable
    w_min = min((float(rt.w[rt.support].min()) for (rt, _) in ora.values() if rt.support.size), default=1.0)

    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, K, kbar, qbar, stride)
    dQ2 = torch.full_like(Q, float("nan"))
    dK = torch.full((w.batch, w.seq, w.h_kv, w.head_dim), float("nan"), device=DEV)
    dV = torch.full_like(dK, float("nan"))
    cap = max(B.dash_attn_list_capacity(p), 1)
    dbias = torch.full((cap,), float("nan"), device=DEV)
    if tensor_cores:
        bws = B.alloc_bwd_workspace(p)
        B.dash_attn_bwd_attend_prefill_tc(p, Q, K, V, dO, mask, bias, dQ2, dK, dV, dbias, bws)
        assert B.dash_attn_last_status(bws) == 0
    else:
        B.dash_attn_bwd_attend_prefill(p, Q, K, V, dO, mask, bias, dQ2, dK, dV, dbias)
    dQr = torch.full((w.batch, w.seq, w.h_q, w.head_dim), float("nan"), device=DEV)
    dKbar = torch.full_like(kbar, float("nan"))
    B.dash_attn_bwd_select_prefill(p, Q, kbar, count, idx, tau, dbias, dQr, dKbar)
    dqbar = None if qbar is None else torch.full_like(qbar, float("nan"))
    B.dash_attn_bwd_block_summaries(p, K, dKbar, dK, qbar, stride, dqbar)
    torch.cuda.synchronize()
    fp32 = Q.dtype == torch.float32
    dQ = dQ2.float().cpu().double().numpy() + dQr.cpu().double().numpy()
    rel = 5e-4 / max(w_min, 1e-3) ** 0.5
    tc = 1e-2 if tensor_cores else 0.0          # P, dS and delta carry bf16 rounding on the tensor-core path
    _close(dQ, ref["dQ"], (2e-3 if fp32 else 1e-2) + rel + tc, "dQ (Stage 2 + routing)")
    _close(dK.cpu().double().numpy(), ref["dK"], 2e-3 + rel + tc, "dK (Stage 2 + summaries)")
    _close(dV.cpu().double().numpy(), ref["dV"], 2e-4 + tc, "dV")
    if qbar is not None:
        _close(dqbar.cpu().double().numpy(), ref["dqbar"], 2e-3 + rel + tc, "dqbar")
    # the routing part alone is not negligible on these inputs (the test would pass trivially otherwise)
    fixed = bwd.backward_prefill(Qn, Kn, Vn, Gn, qbar=qb64, through_routing=False, **kwo)
    if w.seq > 4 * w.block:
        assert np.abs(ref["dQ"] - fixed["dQ"]).max() > 1e-3 * np.abs(ref["dQ"]).max()
        _close(dQr.cpu().double().numpy(), ref["dQ"] - fixed["dQ"], 2e-3 + rel + tc, "dQ through the routing")
