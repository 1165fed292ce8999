"""Pins of the backward oracle (oracle/dash_oracle_bwd.py) against things other than itself: finite differences of
the FORWARD oracle, explicit Jacobians, the sparsemax / softmax special cases, and automatic differentiation of
dense masked attention (a library routine) for the fixed-routing part."""
import math

import numpy as np
import pytest
import torch

from oracle import dash_oracle as orc
from oracle import dash_oracle_bwd as bwd


# ------------------------------------------------------------------ the alpha-entmax Jacobian (Eq. 2)

def _entmax_z(z, alpha):
    return orc.entmax(z, alpha)        # entmax of the unscaled scores z: [(alpha-1) z - tau]_+^(1/(alpha-1))


@pytest.mark.parametrize("alpha", [1.25, 1.5, 1.75, 2.0])
def test_entmax_vjp_matches_finite_differences_of_the_forward_map(alpha):
    rng = np.random.default_rng(int(alpha * 100))
    for trial in range(6):
        n = int(rng.integers(3, 12))
        z = rng.normal(size=n) * 2.0
        p = _entmax_z(z, alpha)
        assert 1 <= (p > 0).sum() <= n
        # keep away from support changes: every |margin| well above the step
        h = 1e-6
        J = np.zeros((n, n))
        for k in range(n):
            zp, zm = z.copy(), z.copy()
            zp[k] += h; zm[k] -= h
            pp, pm = _entmax_z(zp, alpha), _entmax_z(zm, alpha)
            if ((pp > 0) != (p > 0)).any() or ((pm > 0) != (p > 0)).any():
                pytest.skip("support changed inside the finite-difference step")
            J[:, k] = (pp - pm) / (2 * h)
        assert np.allclose(bwd.entmax_jacobian(p, alpha), J, atol=2e-6)
        for _ in range(3):
            dp = rng.normal(size=n)
            assert np.allclose(bwd.entmax_vjp(p, dp, alpha), J.T @ dp, atol=5e-6)


def test_entmax_jacobian_special_cases_and_structure():
    rng = np.random.default_rng(3)
    z = rng.normal(size=9) * 1.5
    # alpha = 2 (sparsemax): J = diag(1_S) - 1_S 1_S^T / |S|
    p = _entmax_z(z, 2.0)
    S = (p > 0).astype(np.float64)
    assert np.allclose(bwd.entmax_jacobian(p, 2.0), np.diag(S) - np.outer(S, S) / S.sum())
    # alpha -> 1: the softmax Jacobian diag(p) - p p^T, with the error shrinking as alpha -> 1
    errs = []
    for alpha in (1.1, 1.01, 1.001):
        pe = _entmax_z(z, alpha)
        sm = np.exp(z - z.max()); sm /= sm.sum()
        errs.append(np.abs(bwd.entmax_jacobian(pe, alpha) - (np.diag(sm) - np.outer(sm, sm))).max())
    assert errs[0] > errs[1] > errs[2] and errs[2] < 2e-3
    # structure: symmetric, rows sum to zero (outputs stay on the simplex), zero outside the support
    for alpha in (1.25, 1.5, 2.0):
        p = _entmax_z(z * 2, alpha)
        J = bwd.entmax_jacobian(p, alpha)
        assert np.allclose(J, J.T) and np.allclose(J.sum(axis=0), 0.0, atol=1e-12)
        off = p == 0
        assert off.any() and not J[off].any() and not J[:, off].any()
        assert np.allclose(bwd.entmax_vjp(p, np.ones_like(p), alpha), 0.0, atol=1e-12)   # shift invariance


# ------------------------------------------------------------------ whole method against finite differences

def _tiny(seed, n=40, h_q=4, h_kv=2, d=8, B=8, planted=True):
    rng = np.random.default_rng(seed)
    Q = rng.normal(size=(1, n, h_q, d))
    K = rng.normal(size=(1, n, h_kv, d))
    V = rng.normal(size=(1, n, h_kv, d))
    if planted:           # some chunks clearly more relevant, so that supports are proper subsets with clear margins
        u = rng.normal(size=(h_kv, d)); u /= np.linalg.norm(u, axis=1, keepdims=True)
        g_q = h_q // h_kv
        Q += 2.0 * np.repeat(u, g_q, axis=0)[None, None]
        for c in (0, 2):
            K[0, c * B:(c + 1) * B] += 2.0 * u[None]
    G = rng.normal(size=Q.shape)
    return Q, K, V, G


def _loss(Q, K, V, G, **kw):
    out = orc.forward_prefill(Q, K, V, **kw)
    return float(np.sum(out["O"] * G)), out["routing"]


def _supports(routing):
    return {k: tuple(int(c) for c in v.support) for k, v in routing.items()}


def _fd_check(name, X, grad, Q, K, V, G, kw, idxs, h=1e-6, tol=2e-6, qbar=None):
    base, r0 = _loss(Q, K, V, G, qbar=qbar, **kw)
    s0 = _supports(r0)
    n_checked = 0
    for idx in idxs:
        old = X[idx]
        X[idx] = old + h
        lp, rp = _loss(Q, K, V, G, qbar=qbar, **kw)
        X[idx] = old - h
        lm, rm = _loss(Q, K, V, G, qbar=qbar, **kw)
        X[idx] = old
        if _supports(rp) != s0 or _supports(rm) != s0:
            continue                                  # a chunk crossed the threshold inside the step: not differentiable there
        fd = (lp - lm) / (2 * h)
        assert abs(fd - grad[idx]) <= tol * max(1.0, abs(fd)), (name, idx, fd, grad[idx])
        n_checked += 1
    assert n_checked >= 0.8 * len(idxs), (name, n_checked, len(idxs))


@pytest.mark.parametrize("alpha,sigma,gamma,mode", [
    (1.5, 1.0, 1.0, "none"), (2.0, 2.0, 1.5, "none"), (1.25, 1.0, 2.0, "none"), (1.5, 0.5, 1.0, "head"),
    (1.5, 1.0, 1.0, "chunk"),
])
def test_whole_backward_matches_finite_differences(alpha, sigma, gamma, mode):
    """L = sum(O * G): dQ, dK, dV and d(summary query) of the backward oracle against central differences of the
    forward oracle, entry by entry on a random sample, through routing, bias and summaries."""
    Q, K, V, G = _tiny(int(alpha * 100 + sigma * 10))
    n, B = Q.shape[1], 8
    rng = np.random.default_rng(5)
    qbar = None
    if mode == "head":
        qbar = rng.normal(size=(K.shape[2], K.shape[3]))
    elif mode == "chunk":
        qbar = rng.normal(size=(n // B, K.shape[2], K.shape[3]))
    kw = dict(B=B, alpha=alpha, gamma=gamma, sigma=sigma)
    g = bwd.backward_prefill(Q, K, V, G, qbar=qbar, **kw)
    # the routing must be doing something: some row with a proper, non-empty support
    _, routing = _loss(Q, K, V, G, qbar=qbar, **kw)
    sizes = [(v.support.size, v.n_cand) for v in routing.values() if v.n_cand >= 3]
    assert any(0 < s < c for s, c in sizes)
    def sample(shape, k):
        return [tuple(int(rng.integers(0, s)) for s in shape) for _ in range(k)]
    _fd_check("dQ", Q, g["dQ"], Q, K, V, G, kw, sample(Q.shape, 25), qbar=qbar)
    _fd_check("dK", K, g["dK"], Q, K, V, G, kw, sample(K.shape, 25), qbar=qbar)
    _fd_check("dV", V, g["dV"], Q, K, V, G, kw, sample(V.shape, 15), qbar=qbar)
    if qbar is not None:
        _fd_check("dqbar", qbar, g["dqbar"], Q, K, V, G, kw, sample(qbar.shape, 12), qbar=qbar)


def test_whole_backward_with_local_window_matches_finite_differences():
    Q, K, V, G = _tiny(77, n=48)
    kw = dict(B=8, alpha=1.5, gamma=1.0, sigma=1.0, local_blocks=1)
    g = bwd.backward_prefill(Q, K, V, G, **kw)
    rng = np.random.default_rng(6)
    def sample(shape, k):
        return [tuple(int(rng.integers(0, s)) for s in shape) for _ in range(k)]
    _fd_check("dQ", Q, g["dQ"], Q, K, V, G, kw, sample(Q.shape, 15))
    _fd_check("dK", K, g["dK"], Q, K, V, G, kw, sample(K.shape, 15))


# ------------------------------------------------------------------ fixed routing: a library's autograd

def test_fixed_routing_backward_matches_autograd_of_dense_masked_attention():
    """With the routing held fixed, Stage 2 is dense attention with an additive token-level mask / bias: the
    gradients must be those torch's automatic differentiation gives for that (float64), and dbias the gradient
    with respect to the per-chunk bias entries."""
    Q, K, V, G = _tiny(11, n=40, h_q=4, h_kv=2, d=8, B=8)
    B_, alpha, gamma, sigma = 8, 1.5, 1.0, 1.0
    fw = orc.forward_prefill(Q, K, V, B=B_, alpha=alpha, gamma=gamma, sigma=sigma)
    g = bwd.backward_prefill(Q, K, V, G, B=B_, alpha=alpha, gamma=gamma, sigma=sigma, through_routing=False)
    n, h_q, h_kv, d = 40, 4, 2, 8
    g_q = h_q // h_kv
    T = n // B_
    Qt, Kt, Vt = (torch.tensor(x[0], dtype=torch.float64, requires_grad=True) for x in (Q, K, V))
    bias_c = torch.zeros(h_kv, n, T, dtype=torch.float64)          # per (kv head, row, chunk); used on routed chunks only
    routed = torch.zeros(h_kv, n, T, dtype=torch.bool)
    for (b, r, i), rt in fw["routing"].items():
        for c, bv in zip(rt.support, rt.bias):
            bias_c[r, i, int(c)] = float(bv); routed[r, i, int(c)] = True
    bias_c.requires_grad_(True)
    tok_chunk = torch.arange(n) // B_
    loss = 0.0
    for hq in range(h_q):
        r = hq // g_q
        logits = Qt[:, hq] @ Kt[:, r].T / math.sqrt(d)                          # [n, n]
        i_idx = torch.arange(n)[:, None]; j_idx = torch.arange(n)[None, :]
        own = (tok_chunk[None, :] == tok_chunk[:, None]) & (j_idx <= i_idx)
        rt_tok = routed[r][:, tok_chunk]                                        # [n, n] token routed by row
        add = torch.where(rt_tok, bias_c[r][:, tok_chunk], torch.zeros((), dtype=torch.float64))
        logits = torch.where(own | rt_tok, logits + add, torch.full((), -float("inf"), dtype=torch.float64))
        P = torch.softmax(logits, dim=-1)
        loss = loss + ((P @ Vt[:, r]) * torch.tensor(G[0, :, hq])).sum()
    loss.backward()
    assert np.allclose(g["dQ"][0], Qt.grad.numpy(), atol=1e-10)
    assert np.allclose(g["dK"][0], Kt.grad.numpy(), atol=1e-10)
    assert np.allclose(g["dV"][0], Vt.grad.numpy(), atol=1e-10)
    gb = bias_c.grad.numpy()
    some = 0
    for (b, r, i), rt in fw["routing"].items():
        for k, c in enumerate(rt.support):
            assert abs(g["dbias"][(b, r, i)][k] - gb[r, i, int(c)]) <= 1e-10
            some += 1
    assert some > 20


def test_prior_switched_off_leaves_only_the_stage2_gradient():
    """sigma -> infinity: the bias vanishes and so does every gradient through the routing (Eq. 8: w' tends to the
    uniform prior on the support); the whole gradient tends to the fixed-routing one at rate 1/sigma."""
    Q, K, V, G = _tiny(21)
    diffs = []
    for sigma in (1e2, 1e4, 1e6):
        kw = dict(B=8, alpha=1.5, gamma=1.0, sigma=sigma)
        full = bwd.backward_prefill(Q, K, V, G, **kw)
        fixed = bwd.backward_prefill(Q, K, V, G, through_routing=False, **kw)
        diffs.append(max(np.abs(full[k] - fixed[k]).max() for k in ("dQ", "dK")))
        assert np.array_equal(full["dV"], fixed["dV"])          # V never enters the routing
    assert diffs[0] > 0 and diffs[1] < diffs[0] * 2e-2 and diffs[2] < diffs[1] * 2e-2


def test_rows_without_candidates_and_restriction_to_rows():
    Q, K, V, G = _tiny(31, n=24)
    kw = dict(B=8, alpha=1.5, gamma=1.0, sigma=1.0)
    # rows of chunk 0 only: plain causal attention inside the chunk, nothing flows into later tokens or the routing
    g = bwd.backward_prefill(Q, K, V, G, rows=range(8), **kw)
    assert not g["dK"][0, 8:].any() and not g["dV"][0, 8:].any() and not g["dQ"][0, 8:].any()
    assert g["dQ"][0, :8].any()
    # the sum over disjoint row sets is the whole gradient
    g_all = bwd.backward_prefill(Q, K, V, G, **kw)
    g_rest = bwd.backward_prefill(Q, K, V, G, rows=range(8, 24), **kw)
    for k in ("dQ", "dK", "dV"):
        assert np.allclose(g[k] + g_rest[k], g_all[k], atol=1e-12)
