"""GPU parity: every stage of the CUDA library, through the C ABI, against the float64 oracle on the same
seeded inputs.  Integer outputs (mask, count, lists) must match exactly except for chunks whose oracle
margin is within 1e-4 of the entmax threshold; floating outputs within the stated tolerances."""
import math

import numpy as np
import pytest
import torch

from oracle import dash_oracle as orc
from paper_2605_18753_b200 import binding as B
from paper_2605_18753_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _wl(**kw):
    base = dict(name="t", kind="prefill", batch=1, seq=512, h_q=4, h_kv=2, head_dim=64, block=16, alpha=1.5,
                dtype="bf16", recipe="planted", gamma=1.0, sigma=10.0, rho=0.72, shift=2.0, n_planted=3, seed=0)
    base.update(kw)
    return synth.Workload(**base)


# ------------------------------------------------------------------ Stage 0

@pytest.mark.parametrize("dtype,d,Bk,n,mode", [
    ("bf16", 128, 64, 1000, "none"), ("bf16", 128, 64, 1000, "head"), ("bf16", 64, 16, 200, "chunk"),
    ("f32", 64, 64, 1024, "none"), ("f32", 128, 128, 700, "head"), ("bf16", 128, 32, 96, "chunk"),
])
def test_block_summaries(dtype, d, Bk, n, mode):
    w = _wl(seq=n, head_dim=d, block=Bk, dtype=dtype, h_q=6, h_kv=3, batch=2)
    inp = synth.make_prefill_inputs(w, DEV)
    K = inp["K"]
    T_s = n // Bk
    qbar = None
    stride = 0
    if mode == "head":
        qbar = torch.randn(3, d, device=DEV, generator=torch.Generator(DEV).manual_seed(5)) * 2
    elif mode == "chunk":
        qbar = torch.randn(T_s, 3, d, device=DEV, generator=torch.Generator(DEV).manual_seed(6)) * 2
        stride = 3 * d
    O = torch.empty_like(inp["Q"])
    p = B.params_for_prefill(inp["Q"], K, inp["V"], O, block=Bk, alpha=1.5)
    kbar = torch.full((2, 3, T_s, d), float("nan"), device=DEV)
    B.dash_attn_block_summaries(p, K, kbar, qbar, stride)
    got = kbar.cpu().double().numpy()
    for bb in range(2):
        want = orc.block_summaries(H.to_np64(K[bb]), Bk, None if qbar is None else H.to_np64(qbar))
        err = np.abs(got[bb].transpose(1, 0, 2) - want)
        assert err.max() <= 2e-6 * max(1.0, np.abs(want).max()), err.max()


def test_block_summaries_incremental_and_kv_len():
    w = _wl(seq=640, head_dim=128, block=64, h_q=2, h_kv=2, batch=2)
    inp = synth.make_prefill_inputs(w, DEV)
    p = B.params_for_prefill(inp["Q"], inp["K"], inp["V"], torch.empty_like(inp["Q"]), block=64, alpha=1.5)
    full = torch.zeros(2, 2, 10, 128, device=DEV)
    B.dash_attn_block_summaries(p, inp["K"], full)
    part = torch.full_like(full, -7.0)
    kv_len = torch.tensor([640, 200], dtype=torch.int32, device=DEV)
    B.dash_attn_block_summaries(p, inp["K"], part, kv_len=kv_len, first_block=2, num_blocks=5)
    assert torch.equal(part[0, :, 2:7], full[0, :, 2:7]) and (part[0, :, :2] == -7).all() and (part[0, :, 7:] == -7).all()
    assert torch.equal(part[1, :, 2:3], full[1, :, 2:3]) and (part[1, :, 3:] == -7).all()   # chunk 3 incomplete at 200


# ------------------------------------------------------------------ Stage 1

def _run_select(w, inp, with_idx=True, local_blocks=0):
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    O = torch.empty_like(Q)
    p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma,
                             local_blocks=local_blocks)
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, K, kbar)
    ws = B.alloc_workspace(p)
    rt = B.alloc_routing(p, with_tau=True)
    for t in rt.values():
        if t is not None:
            t.fill_(-1 if t.dtype != torch.float32 else float("nan"))
    B.dash_attn_select(p, Q, kbar, rt["mask"], rt["count"], rt["blk_idx"] if with_idx else None, rt["blk_bias"], ws,
                       tau=rt["tau"])
    assert B.dash_attn_last_status(ws) == 0
    return p, kbar, ws, rt


def _check_select(w, inp, p, rt, rows, kv_heads=None, local_blocks=0):
    ora = H.oracle_prefill_rows(inp["Q"], inp["K"], inp["V"], B=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma,
                                rows=rows, kv_heads=kv_heads, local_blocks=local_blocks)
    mask = rt["mask"].cpu().numpy().view(np.uint32)
    count = rt["count"].cpu().numpy()
    idx = rt["blk_idx"].cpu().numpy()
    bias = rt["blk_bias"].cpu().numpy()
    tau = rt["tau"].cpu().numpy()
    g_q = w.h_q // w.h_kv
    n_border = n_diff = 0
    clean_rows = {}
    for (b, r, i), (ro, o) in ora.items():
        off = B.dash_attn_list_offset(p, b, r, i)
        nb, nd, clean = H.compare_routing(ro, i // w.block, mask[b, r, i], int(count[b, r, i]), bias[off:], idx[off:],
                                          w.sigma, 1.0 / (w.alpha - 1.0))
        n_border += nb
        n_diff += nd
        clean_rows[(b, r, i)] = clean
        if ro.n_cand:
            terr = np.abs(tau[b, r * g_q:(r + 1) * g_q, i] - ro.tau).max()
            assert terr <= 1e-5 * max(1.0, np.abs(ro.x).max()), (i, terr)
    return ora, clean_rows, n_border, n_diff


@pytest.mark.parametrize("kw", [
    dict(), dict(alpha=2.0), dict(alpha=1.25, gamma=2.0), dict(alpha=1.75, gamma=1.5),
    dict(h_q=8, h_kv=2, head_dim=128, block=32, seq=1000), dict(h_q=2, h_kv=2, block=64, seq=777),
    dict(h_q=16, h_kv=1, head_dim=128, block=64, seq=1500, batch=2), dict(dtype="f32", seq=300, gamma=3.0),
    dict(h_q=8, h_kv=1, head_dim=64, block=128, seq=1100), dict(seq=15), dict(seq=16), dict(seq=17),
    dict(h_q=8, h_kv=1, head_dim=128, block=16, seq=9000),      # rows beyond 512 candidates: clusters of two blocks
    dict(h_q=16, h_kv=1, head_dim=128, block=16, seq=17000, n_planted=6),   # beyond 1024: clusters of four
    dict(h_q=4, h_kv=2, head_dim=128, block=64, seq=2100, alpha=2.0), dict(h_q=32, h_kv=2, head_dim=128, block=32, seq=700),
    dict(h_q=4, h_kv=1, head_dim=128, block=16, seq=9000),      # tiles of 16 tokens (64 live rows) in clusters of two blocks
    dict(h_q=4, h_kv=2, head_dim=64, block=32, seq=3000, alpha=1.25),   # g_q = 2: tiles of 32 tokens, head_dim 64
])
def test_select_matches_oracle(kw):
    w = _wl(**kw)
    inp = synth.make_prefill_inputs(w, DEV)
    p, kbar, ws, rt = _run_select(w, inp)
    step = 7 if w.seq < 12000 else 41
    rows = sorted(set(list(range(0, w.seq, step)) + [w.seq - 1] + list(range(min(w.seq, 3 * w.block)))))
    ora, clean, nb, nd = _check_select(w, inp, p, rt, rows)
    sizes = [v[0].support.size for v in ora.values()]
    if w.seq > 4 * w.block:
        assert max(sizes) >= 2
    assert nd <= nb


def test_select_tiny_configs_and_sparsity_regimes():
    """C1 (gamma=1: every visible chunk routed) and C1' (gamma=512: the threshold prunes), fp32."""
    for name in ("tiny", "tiny_g512"):
        w = synth.workload(name)
        inp = synth.make_prefill_inputs(w, DEV)
        p, kbar, ws, rt = _run_select(w, inp)
        ora, clean, nb, nd = _check_select(w, inp, p, rt, range(w.seq))
        sup = [v[0].support.size for v in ora.values()]
        vis = [i // w.block for (_, _, i) in ora.keys()]
        s = orc.block_sparsity(sup, vis)
        assert (s == 0.0) if name == "tiny" else (0.3 < s < 0.6)


def test_select_without_block_index_list_and_determinism():
    w = _wl(seq=900, h_q=8, h_kv=2, head_dim=128, block=64)
    inp = synth.make_prefill_inputs(w, DEV)
    p, kbar, ws, rt1 = _run_select(w, inp, with_idx=True)
    p, kbar, ws, rt2 = _run_select(w, inp, with_idx=False)
    assert torch.equal(rt1["mask"], rt2["mask"]) and torch.equal(rt1["count"], rt2["count"])
    assert torch.equal(rt1["tau"], rt2["tau"])
    assert (rt2["blk_idx"] == -1).all()


# ------------------------------------------------------------------ Stage 2 (prefill)

def _gather_O(O, keys, g_q):
    On = O.float().cpu().double().numpy()
    return np.stack([On[b, i, r * g_q:(r + 1) * g_q] for (b, r, i) in keys])


@pytest.mark.parametrize("kw", [
    dict(), dict(dtype="f32"), dict(h_q=8, h_kv=2, head_dim=128, block=64, seq=1000, sigma=1.0),
    dict(h_q=4, h_kv=4, head_dim=128, block=32, seq=333, alpha=2.0), dict(seq=17), dict(seq=5),
    dict(h_q=16, h_kv=1, head_dim=128, block=128, seq=700, alpha=1.25, gamma=2.0),
    dict(h_q=8, h_kv=2, head_dim=128, block=32, seq=900, gamma=2.0),     # packed chunks (two per step), every row compared
    dict(h_q=8, h_kv=1, head_dim=64, block=16, seq=500, gamma=2.0),      # four per step, head_dim 64
    dict(h_q=4, h_kv=2, head_dim=128, block=16, seq=400, gamma=2.0),     # short tiles (32 live rows)
])
def test_attend_prefill_with_oracle_lists(kw):
    """Stage 2 alone, fed the oracle's own routing: no exclusions, every row must match."""
    w = _wl(**kw)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    O = torch.full_like(Q, float("nan"))
    p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    ora = H.oracle_prefill_rows(Q, K, V, B=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, rows=range(w.seq))
    mask, count, idx, bias = H.routing_to_abi(ora, p, B.dash_attn_list_offset)
    ws = B.alloc_workspace(p)
    B.dash_attn_attend_prefill(p, Q, K, V, mask, bias, O, ws)
    assert B.dash_attn_last_status(ws) == 0
    keys = list(ora.keys())
    want = np.stack([ora[k][1] for k in keys])
    H.check_outputs(_gather_O(O, keys, w.h_q // w.h_kv), want, Q.dtype, "attend_prefill")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_attend_prefill_running_maximum_moves_late(dtype):
    """Keys whose magnitude rises from chunk to chunk in periods of five: along a row's walk (own chunk first, then its
    routed chunks in ascending order) the row maximum grows by more than the lazy-rescale threshold several times, so
    the accumulator is rescaled in tensor memory well after its first products.  Stage 2 alone on the oracle's lists,
    every row compared."""
    w = _wl(seq=900, h_q=8, h_kv=2, head_dim=128, block=64, gamma=0.1, dtype=dtype)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    fac = 1.0 + 2.5 * ((torch.arange(w.seq, device=DEV) // w.block) % 5).float()
    K = (K.float() * fac[None, :, None, None]).to(K.dtype)
    O = torch.full_like(Q, float("nan"))
    p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    ora = H.oracle_prefill_rows(Q, K, V, B=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, rows=range(w.seq))
    # the premise: on a sample of rows, count the steps at which the maximum grows by more than 2^8
    Qn, Kn = H.to_np64(Q), H.to_np64(K)
    g_q, c1 = w.h_q // w.h_kv, 1.4426950408889634 / np.sqrt(w.head_dim)
    moves = []
    for (b, r, i), (rt, _) in list(ora.items())[::9]:
        q = Qn[b, i, r * g_q]
        m = (Kn[b, (i // w.block) * w.block:i + 1, r] @ q).max() * c1
        k = 0
        for c, bias in zip(rt.support, rt.bias):
            mm = (Kn[b, int(c) * w.block:(int(c) + 1) * w.block, r] @ q).max() * c1 + bias * 1.4426950408889634
            if mm > m + 8.0:
                m, k = mm, k + 1
        moves.append(k)
    assert np.mean(np.array(moves) >= 2) > 0.2, np.bincount(moves)
    mask, count, idx, bias = H.routing_to_abi(ora, p, B.dash_attn_list_offset)
    ws = B.alloc_workspace(p)
    B.dash_attn_attend_prefill(p, Q, K, V, mask, bias, O, ws)
    assert B.dash_attn_last_status(ws) == 0
    keys = list(ora.keys())
    want = np.stack([ora[k][1] for k in keys])
    H.check_outputs(_gather_O(O, keys, g_q), want, Q.dtype, "attend_prefill, late maxima")


@pytest.mark.parametrize("name,sigmas", [("tiny", (10.0, 1.0, 1e8)), ("tiny_g512", (10.0, 1e8))])
def test_fwd_prefill_tiny_fp32(name, sigmas):
    for sigma in sigmas:
        w = synth.workload(name, sigma=sigma)
        _fwd_prefill_case(w, rows=range(w.seq))


@pytest.mark.parametrize("kw", [
    dict(seq=1024, h_q=8, h_kv=2, head_dim=128, block=64),
    dict(seq=1024, h_q=8, h_kv=2, head_dim=128, block=64, sigma=1e8),
    dict(seq=2000, h_q=4, h_kv=1, head_dim=128, block=128, alpha=2.0, batch=2),
    dict(seq=600, h_q=4, h_kv=2, head_dim=64, block=32, alpha=1.25, gamma=2.0),
    dict(seq=1500, h_q=32, h_kv=2, head_dim=128, block=64, seed=1),
    dict(seq=1111, h_q=2, h_kv=2, head_dim=128, block=64, seed=2),
    dict(seq=1300, h_q=16, h_kv=2, head_dim=128, block=64, seed=3),          # g_q = 8 on the tensor-core paths
    dict(seq=900, h_q=4, h_kv=2, head_dim=128, block=128, seed=4),           # g_q = 2, chunks of 128
    dict(seq=1500, h_q=8, h_kv=2, head_dim=64, block=64, seed=6),            # head_dim 64 on the tensor-core kernels
    dict(seq=1100, h_q=16, h_kv=1, head_dim=64, block=128, seed=7, alpha=2.0),
    dict(seq=1300, h_q=8, h_kv=2, head_dim=128, block=32, seed=8),           # two chunks of 32 per 64-token step
    dict(seq=1000, h_q=16, h_kv=2, head_dim=128, block=16, seed=9),          # four chunks of 16 per step (g_q = 8)
    dict(seq=777, h_q=16, h_kv=1, head_dim=64, block=16, seed=10, alpha=1.25, gamma=2.0),
    dict(seq=2100, h_q=4, h_kv=2, head_dim=128, block=32, seed=11, n_planted=6),   # g_q = 2, chunks of 32: tiles of 32 tokens, 64 live rows
    dict(seq=1500, h_q=8, h_kv=2, head_dim=128, block=16, seed=12),                # g_q = 4, chunks of 16: tiles of 16 tokens
    dict(seq=900, h_q=2, h_kv=1, head_dim=64, block=16, seed=13, alpha=2.0),        # g_q = 2, chunks of 16: 32 live rows
])
def test_fwd_prefill_small(kw):
    w = _wl(**kw)
    rows = sorted(set(list(range(0, w.seq, 5)) + [w.seq - 1, w.seq - 2] + list(range(min(w.seq, 2 * w.block)))))
    _fwd_prefill_case(w, rows)


def _fwd_prefill_case(w, rows, kv_heads=None, min_clean=0.9, local_blocks=0, qbar_mode="none", give_kbar=False):
    """qbar_mode: "none" (mean pooling), "head" (one summary query per KV head), "chunk" (one per chunk and KV head);
    give_kbar: the caller computes the summaries with dash_attn_block_summaries and hands them to the forward."""
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    O = torch.full_like(Q, float("nan"))
    p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma,
                             local_blocks=local_blocks)
    ws = B.alloc_workspace(p)
    T_a = (w.seq + w.block - 1) // w.block
    T_s = w.seq // w.block
    mask = torch.empty(w.batch, w.h_kv, w.seq, (T_a + 31) // 32, dtype=torch.int32, device=DEV)
    qbar, stride = None, 0
    if qbar_mode == "head":
        qbar = torch.randn(w.h_kv, w.head_dim, device=DEV, generator=torch.Generator(DEV).manual_seed(w.seed + 50)) * 2
    elif qbar_mode == "chunk":
        qbar = torch.randn(max(T_s, 1), w.h_kv, w.head_dim, device=DEV,
                           generator=torch.Generator(DEV).manual_seed(w.seed + 51)) * 2
        stride = w.h_kv * w.head_dim
    if give_kbar:
        kbar = B.alloc_kbar(p)
        B.dash_attn_block_summaries(p, K, kbar, qbar, stride)
        B.dash_attn_fwd_prefill(p, Q, K, V, O, ws, Kbar=kbar, mask_out=mask)
    else:
        B.dash_attn_fwd_prefill(p, Q, K, V, O, ws, qbar=qbar, qbar_chunk_stride=stride, mask_out=mask)
    assert B.dash_attn_last_status(ws) == 0
    assert torch.isfinite(O.float()).all()
    ora = H.oracle_prefill_rows(Q, K, V, B=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, rows=rows,
                                kv_heads=kv_heads, local_blocks=local_blocks,
                                qbar=None if qbar is None else H.to_np64(qbar))
    mk = mask.cpu().numpy().view(np.uint32)
    keys = []
    n_excluded = 0
    for (b, r, i), (ro, o) in ora.items():
        want = orc.pack_mask_words(np.concatenate([ro.support, ro.local]), i // w.block, mk.shape[-1])
        if np.array_equal(mk[b, r, i], want):
            # rows holding a member or non-member inside the borderline band are compared on the mask only:
            # at finite sigma their bias (log of a near-zero weight) is ill-conditioned by construction
            if ro.n_cand and (np.abs(ro.margin) <= H.BORDERLINE).any():
                n_excluded += 1
            else:
                keys.append((b, r, i))
        else:
            got = {c for c in range(T_a) if (int(mk[b, r, i, c >> 5]) >> (c & 31)) & 1}
            diff = got ^ (set(int(c) for c in ro.support) | set(int(c) for c in ro.local) | {i // w.block})
            border = set(int(c) for c in np.nonzero(np.abs(ro.margin) <= H.BORDERLINE)[0])
            assert diff <= border, (b, r, i, sorted(diff))
            n_excluded += 1
    assert len(keys) >= min_clean * len(ora), f"too few clean rows: {len(keys)} of {len(ora)} ({n_excluded} excluded)"
    want = np.stack([ora[k][1] for k in keys])
    return H.check_outputs(_gather_O(O, keys, w.h_q // w.h_kv), want, Q.dtype, f"fwd_prefill {w.name}")


@pytest.mark.parametrize("kw,qbar_mode,give_kbar", [
    (dict(seq=1024, h_q=8, h_kv=2, head_dim=128, block=64, seed=20), "head", False),    # planes written by Stage 0, weighted
    (dict(seq=1100, h_q=8, h_kv=2, head_dim=128, block=64, seed=21), "chunk", False),
    (dict(seq=900, h_q=16, h_kv=2, head_dim=64, block=32, seed=22, alpha=2.0), "chunk", False),
    (dict(seq=700, dtype="f32", gamma=3.0, seed=23), "head", False),                    # CUDA-core path
    (dict(seq=1024, h_q=8, h_kv=2, head_dim=128, block=64, seed=24), "none", True),     # caller-supplied summaries
    (dict(seq=1300, h_q=32, h_kv=2, head_dim=128, block=64, seed=25), "head", True),
])
def test_fwd_prefill_with_summary_queries_and_given_summaries(kw, qbar_mode, give_kbar):
    """The whole forward with a learned summary query (Eq. 3: softmax-weighted pooling, per KV head or per chunk as
    Algorithm 1's input) and with summaries the caller computed beforehand."""
    w = _wl(**kw)
    rows = sorted(set(list(range(0, w.seq, 5)) + [w.seq - 1, w.seq - 2] + list(range(min(w.seq, 2 * w.block)))))
    _fwd_prefill_case(w, rows, qbar_mode=qbar_mode, give_kbar=give_kbar)


def test_select_equal_scores_get_equal_weights():
    """Duplicated key chunks have identical summaries, hence identical logits: entmax is symmetric, so the copies are
    routed together (or not at all) and carry the same bias; the rest of the routing still matches the oracle."""
    w = _wl(seq=1500, h_q=8, h_kv=2, head_dim=128, block=64, seed=30)
    inp = synth.make_prefill_inputs(w, DEV)
    K = inp["K"]
    pairs = [(1, 9), (3, 17), (4, 5)]
    for a, c in pairs:
        K[:, c * 64:(c + 1) * 64] = K[:, a * 64:(a + 1) * 64]
    p, kbar, ws, rt = _run_select(w, inp)
    assert torch.equal(kbar[:, :, 1], kbar[:, :, 9])
    rows = sorted(set(list(range(0, w.seq, 3)) + [w.seq - 1]))
    _check_select(w, inp, p, rt, rows)
    mask = rt["mask"].cpu().numpy().view(np.uint32)
    count = rt["count"].cpu().numpy()
    idx, bias = rt["blk_idx"].cpu().numpy(), rt["blk_bias"].cpu().numpy()
    n_both = 0
    for r in range(w.h_kv):
        for i in range(18 * 64, w.seq, 3):
            off = B.dash_attn_list_offset(p, 0, r, i)
            ent = {int(c): float(v) for c, v in zip(idx[off:off + count[0, r, i]], bias[off:off + count[0, r, i]])}
            for a, c in pairs:
                assert (a in ent) == (c in ent), (r, i, a, c)
                assert ((mask[0, r, i, a >> 5] >> (a & 31)) & 1) == ((mask[0, r, i, c >> 5] >> (c & 31)) & 1)
                if a in ent:
                    assert ent[a] == ent[c], (r, i, a, c, ent[a], ent[c])
                    n_both += 1
    assert n_both > 0


def test_select_rows_beyond_2048_candidates():
    """Chunks of 16 tokens and more than 32784 tokens: the last rows have more than 2048 candidates, beyond what
    the tensor-core routing kernel keeps on chip; they take the CUDA-core kernel."""
    w = _wl(seq=33100, h_q=2, h_kv=1, head_dim=64, block=16, seed=31, n_planted=6)
    inp = synth.make_prefill_inputs(w, DEV)
    p, kbar, ws, rt = _run_select(w, inp)
    rows = sorted(set(list(range(32784, w.seq, 9)) + list(range(32700, 32784, 7)) + list(range(0, 32700, 997))
                      + [w.seq - 1]))
    ora, clean, nb, nd = _check_select(w, inp, p, rt, rows)
    assert max(v[0].n_cand for v in ora.values()) > 2048
    assert nd <= nb


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_fwd_prefill_8k_config_sampled_rows(seed):
    """The 8K prefill workload at full size, in the configuration the benchmark times (seed 0) and on two more
    seeds; the oracle computes a seeded sample of rows (first/last rows of chunks, random rows, two whole tiles)."""
    w = synth.workload("prefill_8k", seed=seed)
    rng = np.random.default_rng(seed)
    rows = set(rng.integers(0, w.seq, 1024).tolist()) | {0, 63, 64, 65, 127, 128, w.seq - 1, w.seq - 64, w.seq - 65}
    rows |= set(range(4096, 4096 + 32)) | set(range(8000, 8032))
    for sigma in ((10.0, 1e8) if seed == 0 else (10.0,)):
        _fwd_prefill_case(w.with_(sigma=sigma), sorted(rows), kv_heads=[0, 5])


# ------------------------------------------------------------------ decode

def _decode_case(w, kv_len, use_lists_from_oracle=False, local_blocks=0, key_ramp=False):
    inp = synth.make_decode_inputs(w, DEV, kv_len=kv_len)
    Q, Kc, Vc, lens = inp["Q"], inp["K"], inp["V"], inp["kv_len"]
    if key_ramp:      # key magnitudes rise from chunk to chunk in periods of five: partial maxima far apart
        fac = 1.0 + 2.5 * ((torch.arange(Kc.shape[1], device=DEV) // w.block) % 5).float()
        Kc = (Kc.float() * fac[None, :, None, None]).to(Kc.dtype)
    O = torch.full_like(Q, float("nan"))
    p = B.params_for_decode(Q, Kc, Vc, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma,
                            local_blocks=local_blocks)
    kbar = B.alloc_kbar(p)
    kbar.fill_(float("nan"))
    B.dash_attn_block_summaries(p, Kc, kbar, kv_len=lens)
    ws = B.alloc_workspace(p)
    ora = orc.forward_decode(H.to_np64(Q), H.to_np64(Kc), H.to_np64(Vc), lens.cpu().numpy(), B=w.block, alpha=w.alpha,
                             gamma=w.gamma, sigma=w.sigma, local_blocks=local_blocks)
    if use_lists_from_oracle:
        mask, count, idx, bias = H.routing_to_abi({(b, r, 0): rt for (b, r), rt in ora["routing"].items()}, p,
                                                  B.dash_attn_list_offset)
        B.dash_attn_attend_decode(p, Q, Kc, Vc, lens, count, idx, bias, O, ws)
        assert B.dash_attn_last_status(ws) == 0
        H.check_outputs(O.float().cpu().double().numpy(), ora["O"], Q.dtype, "attend_decode")
        return
    # Stage 1 alone on the decode row, then the whole step
    rt = B.alloc_routing(p, with_tau=True)
    B.dash_attn_select(p, Q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws, tau=rt["tau"], kv_len=lens)
    mask = rt["mask"].cpu().numpy().view(np.uint32)
    count = rt["count"].cpu().numpy()
    idx = rt["blk_idx"].cpu().numpy()
    bias = rt["blk_bias"].cpu().numpy()
    clean = np.ones((w.batch, w.h_kv), dtype=bool)
    for (b, r), ro in ora["routing"].items():
        off = B.dash_attn_list_offset(p, b, r, 0)
        L = int(lens[b])
        nb, nd, ok = H.compare_routing(ro, (L - 1) // w.block, mask[b, r, 0], int(count[b, r, 0]), bias[off:], idx[off:],
                                       w.sigma, 1.0 / (w.alpha - 1.0))
        clean[b, r] = ok and not (ro.n_cand and (np.abs(ro.margin) <= H.BORDERLINE).any())
    B.dash_attn_fwd_decode(p, Q, Kc, Vc, kbar, lens, O, ws)
    assert B.dash_attn_last_status(ws) == 0
    got = O.float().cpu().double().numpy()
    g_q = w.h_q // w.h_kv
    sel = np.repeat(clean, g_q, axis=1)
    assert sel.any() and (sel.mean() >= 0.8 or sel.size < 64), "too few clean groups"
    H.check_outputs(got[sel], ora["O"][sel], Q.dtype, "fwd_decode")


@pytest.mark.parametrize("kw,kv_len", [
    (dict(kind="decode", batch=3, seq=2000, h_q=8, h_kv=2, head_dim=128, block=64), [2000, 1, 777]),
    (dict(kind="decode", batch=2, seq=1024, h_q=4, h_kv=4, head_dim=64, block=32, alpha=2.0), [1024, 65]),
    (dict(kind="decode", batch=2, seq=4096, h_q=16, h_kv=1, head_dim=128, block=128, alpha=1.25, gamma=2.0), [4095, 129]),
    (dict(kind="decode", batch=1, seq=3000, h_q=2, h_kv=2, head_dim=128, block=64, dtype="f32"), [2999]),
    (dict(kind="decode", batch=2, seq=5000, h_q=16, h_kv=2, head_dim=128, block=64), [5000, 4097]),     # g_q = 8
    (dict(kind="decode", batch=2, seq=3000, h_q=4, h_kv=2, head_dim=128, block=128, alpha=2.0), [3000, 2050]),   # g_q = 2
    (dict(kind="decode", batch=3, seq=2500, h_q=8, h_kv=2, head_dim=128, block=32), [2500, 33, 1999]),   # two chunks per sub-block
    (dict(kind="decode", batch=2, seq=1800, h_q=16, h_kv=2, head_dim=128, block=16, alpha=1.25, gamma=2.0), [1800, 1001]),
    (dict(kind="decode", batch=2, seq=9000, h_q=4, h_kv=1, head_dim=128, block=16), [9000, 8191]),      # long lists, four per sub-block
    (dict(kind="decode", batch=3, seq=4000, h_q=16, h_kv=2, head_dim=64, block=64), [4000, 1, 2049]),   # head_dim 64: stacked sub-blocks
    (dict(kind="decode", batch=2, seq=3000, h_q=8, h_kv=2, head_dim=64, block=128, alpha=2.0), [2999, 130]),
    (dict(kind="decode", batch=2, seq=2500, h_q=2, h_kv=1, head_dim=64, block=32), [2500, 1777]),
    # more than 2048 candidates: the routing warp keeps 64 logits per lane and re-reads the rest from shared memory
    (dict(kind="decode", batch=2, seq=40000, h_q=4, h_kv=1, head_dim=64, block=16), [40000, 33000]),
])
def test_decode_matches_oracle(kw, kv_len):
    w = _wl(**kw)
    _decode_case(w, kv_len, use_lists_from_oracle=True)
    _decode_case(w, kv_len)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_decode_partial_maxima_far_apart(dtype):
    """Key magnitudes that rise from chunk to chunk: the running maximum of a split moves by more than the lazy-rescale
    threshold several times and the splits of a (batch, KV head) end with maxima tens of units apart, which the merge
    has to bring onto one scale."""
    w = _wl(kind="decode", batch=2, seq=6000, h_q=8, h_kv=2, head_dim=128, block=64, gamma=0.1, dtype=dtype)
    _decode_case(w, [6000, 3100], use_lists_from_oracle=True, key_ramp=True)
    _decode_case(w, [6000, 3100], key_ramp=True)


def test_decode_equals_last_prefill_row_on_gpu():
    w = _wl(seq=1000, h_q=8, h_kv=2, head_dim=128, block=64)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    O = torch.empty_like(Q)
    p = B.params_for_prefill(Q, K, V, O, block=64, alpha=1.5)
    ws = B.alloc_workspace(p)
    B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
    q1 = Q[:, -1].contiguous()
    o1 = torch.empty_like(q1)
    pd = B.params_for_decode(q1, K, V, o1, block=64, alpha=1.5)
    kbar = B.alloc_kbar(pd)
    B.dash_attn_block_summaries(pd, K, kbar)
    wsd = B.alloc_workspace(pd)
    B.dash_attn_fwd_decode(pd, q1, K, V, kbar, None, o1, wsd)
    assert (o1.float() - O[:, -1].float()).abs().max().item() <= 2e-2


# ------------------------------------------------------------------ strided tensors

@pytest.mark.parametrize("layout", ["packed_qkv", "head_major"])
def test_fwd_prefill_and_decode_on_strided_views(layout):
    """Q, K, V, O as views of larger buffers (one packed [b, n, h_q + 2 h_kv, d] projection output; a head-major
    [b, h, n, d] buffer): only the element strides in the parameter block change, the results must not."""
    w = _wl(seq=1200, h_q=8, h_kv=2, head_dim=128, block=64, seed=5)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    O = torch.empty_like(Q)
    p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    ws = B.alloc_workspace(p)
    B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
    assert B.dash_attn_last_status(ws) == 0

    b, n, h_q, h_kv, d = w.batch, w.seq, w.h_q, w.h_kv, w.head_dim
    if layout == "packed_qkv":
        buf = torch.full((b, n, h_q + 2 * h_kv, d), float("nan"), dtype=Q.dtype, device=DEV)
        buf[:, :, :h_q] = Q
        buf[:, :, h_q:h_q + h_kv] = K
        buf[:, :, h_q + h_kv:] = V
        Qs, Ks, Vs = buf[:, :, :h_q], buf[:, :, h_q:h_q + h_kv], buf[:, :, h_q + h_kv:]
        Os = torch.full((b, n, h_q + 3, d), float("nan"), dtype=Q.dtype, device=DEV)[:, :, 3:]
    else:
        Qs = Q.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)       # storage [b, h, n, d], viewed [b, n, h, d]
        Ks = K.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        Vs = V.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        Os = torch.empty(b, h_q, n, d, dtype=Q.dtype, device=DEV).permute(0, 2, 1, 3)
    assert not Qs.is_contiguous() and Qs.stride(-1) == 1
    ps = B.params_for_prefill(Qs, Ks, Vs, Os, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    ws2 = B.alloc_workspace(ps)
    B.dash_attn_fwd_prefill(ps, Qs, Ks, Vs, Os, ws2)
    assert B.dash_attn_last_status(ws2) == 0
    assert torch.equal(Os, O)

    # decode on the same views: the last token against the strided cache
    q1 = Qs[:, -1]
    o1 = torch.empty(b, h_q, d, dtype=Q.dtype, device=DEV)
    pd = B.params_for_decode(q1, Ks, Vs, o1, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(pd)
    B.dash_attn_block_summaries(pd, Ks, kbar)
    wsd = B.alloc_workspace(pd)
    B.dash_attn_fwd_decode(pd, q1, Ks, Vs, kbar, None, o1, wsd)
    assert B.dash_attn_last_status(wsd) == 0
    assert (o1.float() - O[:, -1].float()).abs().max().item() <= 2e-2


# ------------------------------------------------------------------ local window (own chunk + previous chunks)

@pytest.mark.parametrize("kw,L", [
    (dict(), 1), (dict(), 3), (dict(alpha=2.0, seq=300), 2), (dict(dtype="f32", seq=300, gamma=3.0), 1),
    (dict(h_q=8, h_kv=2, head_dim=128, block=32, seq=1000), 1),
    (dict(h_q=16, h_kv=1, head_dim=128, block=64, seq=1500, batch=2), 2),
    (dict(h_q=8, h_kv=1, head_dim=128, block=16, seq=9000), 1),      # clusters of two blocks
    (dict(h_q=32, h_kv=2, head_dim=128, block=32, seq=700), 40),     # window longer than the sequence: nothing routed
    (dict(h_q=4, h_kv=2, head_dim=128, block=64, seq=2100), 31), (dict(h_q=4, h_kv=2, head_dim=128, block=64, seq=2100), 33),
])
def test_select_with_local_window(kw, L):
    w = _wl(**kw)
    inp = synth.make_prefill_inputs(w, DEV)
    p, kbar, ws, rt = _run_select(w, inp, local_blocks=L)
    step = 7 if w.seq < 12000 else 41
    rows = sorted(set(list(range(0, w.seq, step)) + [w.seq - 1] + list(range(min(w.seq, (L + 2) * w.block)))))
    ora, clean, nb, nd = _check_select(w, inp, p, rt, rows, local_blocks=L)
    assert nd <= nb
    assert all(v[0].local.size == min(L, i // w.block) for (b, r, i), v in ora.items())


@pytest.mark.parametrize("kw,L", [
    (dict(seq=640, h_q=8, h_kv=2, head_dim=128, block=64, seed=3), 1),
    (dict(seq=900, h_q=4, h_kv=2, head_dim=128, block=128, seed=4), 2),
    (dict(seq=500, dtype="f32", gamma=3.0), 1),
    (dict(seq=1300, h_q=32, h_kv=2, head_dim=128, block=64, seed=5), 1),
])
def test_fwd_prefill_with_local_window(kw, L):
    w = _wl(**kw)
    rows = sorted(set(list(range(0, w.seq, 5)) + [w.seq - 1, w.seq - 2] + list(range(min(w.seq, 3 * w.block)))))
    _fwd_prefill_case(w, rows, local_blocks=L)


def test_fwd_prefill_8k_config_with_the_training_window():
    """The 8K workload with the window of the paper's trained models (own chunk + previous chunk)."""
    w = synth.workload("prefill_8k")
    rng = np.random.default_rng(7)
    rows = set(rng.integers(0, w.seq, 512).tolist()) | {0, 63, 64, 65, 127, 128, 129, w.seq - 1, w.seq - 64, w.seq - 65}
    _fwd_prefill_case(w, sorted(rows), kv_heads=[1, 6], local_blocks=1)


def test_window_covering_the_sequence_is_dense_causal_attention():
    """Nothing is left to route when the window reaches back to token 0: the forward pass must equal dense causal
    softmax attention (torch SDPA in fp32 on the same bf16 tensors), whatever alpha and sigma are."""
    w = _wl(seq=1000, h_q=8, h_kv=2, head_dim=128, block=64, alpha=1.25, sigma=0.5)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    O = torch.full_like(Q, float("nan"))
    p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, local_blocks=16)
    ws = B.alloc_workspace(p)
    B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
    assert B.dash_attn_last_status(ws) == 0
    q, k, v = (t.float().transpose(1, 2) for t in (Q, K, V))
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True, enable_gqa=True).transpose(1, 2)
    H.check_outputs(O.float().cpu().double().numpy(), ref.cpu().double().numpy(), Q.dtype, "window = everything")


@pytest.mark.parametrize("kw,kv_len,L", [
    (dict(kind="decode", batch=3, seq=2000, h_q=8, h_kv=2, head_dim=128, block=64), [2000, 1, 777], 1),
    (dict(kind="decode", batch=2, seq=5000, h_q=32, h_kv=8, head_dim=128, block=64), [5000, 4097], 2),
    (dict(kind="decode", batch=2, seq=600, h_q=4, h_kv=2, head_dim=64, block=16, dtype="f32"), [600, 33], 3),
    (dict(kind="decode", batch=2, seq=1500, h_q=8, h_kv=2, head_dim=128, block=64), [1500, 130], 50),
])
def test_decode_with_local_window(kw, kv_len, L):
    w = _wl(**kw)
    _decode_case(w, kv_len, local_blocks=L)


# ------------------------------------------------------------------ non-causal reading (CUDA-core kernels)

@pytest.mark.parametrize("kw", [
    dict(seq=200), dict(seq=192), dict(seq=333, dtype="f32", gamma=3.0), dict(seq=15),
    dict(seq=700, h_q=8, h_kv=2, head_dim=128, block=64, alpha=2.0),
    dict(seq=640, h_q=16, h_kv=2, head_dim=128, block=32, alpha=1.25, gamma=2.0, batch=2),
])
def test_non_causal_prefill_matches_oracle(kw):
    """causal = 0: all complete chunks are candidates of every row, the incomplete tail chunk is attended whole
    with bias 0, no causal mask.  Routing lists and outputs against the oracle's non-causal reading."""
    w = _wl(**kw)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    O = torch.full_like(Q, float("nan"))
    p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, causal=0)
    T_s, T_a = w.seq // w.block, (w.seq + w.block - 1) // w.block
    own = T_s if T_a > T_s else None
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, K, kbar)
    ws = B.alloc_workspace(p)
    rt = B.alloc_routing(p, with_tau=True)
    B.dash_attn_select(p, Q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws, tau=rt["tau"])
    assert B.dash_attn_last_status(ws) == 0
    rows = sorted(set(list(range(0, w.seq, 3)) + [w.seq - 1]))
    ora = H.oracle_prefill_rows(Q, K, V, B=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, rows=rows, causal=False)
    mask = rt["mask"].cpu().numpy().view(np.uint32)
    count, idx, bias = rt["count"].cpu().numpy(), rt["blk_idx"].cpu().numpy(), rt["blk_bias"].cpu().numpy()
    clean = {}
    for (b, r, i), (ro, o) in ora.items():
        assert ro.n_cand == T_s
        off = B.dash_attn_list_offset(p, b, r, i)
        assert off == (b * w.h_kv + r) * w.seq * T_s + i * T_s
        nb, nd, ok = H.compare_routing(ro, own, mask[b, r, i], int(count[b, r, i]), bias[off:], idx[off:], w.sigma,
                                       1.0 / (w.alpha - 1.0))
        clean[(b, r, i)] = ok and not (ro.n_cand and (np.abs(ro.margin) <= H.BORDERLINE).any())
    B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
    assert B.dash_attn_last_status(ws) == 0
    keys = [k for k, ok in clean.items() if ok]
    assert len(keys) >= 0.9 * len(ora)
    if T_s == 0:
        assert all(v[0].support.size == 0 for v in ora.values())
    H.check_outputs(_gather_O(O, keys, w.h_q // w.h_kv), np.stack([ora[k][1] for k in keys]), Q.dtype, "non-causal")
