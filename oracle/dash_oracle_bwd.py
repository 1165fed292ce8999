"""Float64 CPU oracle for the DashAttention BACKWARD pass.

TEST INFRASTRUCTURE ONLY, like ``dash_oracle`` (the forward oracle) beside it: plain, slow, by the definition.
It shares no code with the CUDA path and nothing in the product package imports it.

What the paper fixes about the backward pass (Section 3.5, last sentence of the Stage-2 kernel paragraph; appendix
"The alpha-entmax mapping", paragraph on differentiability): the gradient flows from the output through the softmax
refinement into the routed chunks' entmax weights and on into the chunk summaries; the backward kernels reuse the bit
mask of the forward pass because, where the support is fixed, alpha-entmax has a closed-form SPARSE Jacobian (zero
rows and columns outside the support).  The paper prints no backward formulas, so each function below states the
forward relation it differentiates and the derivative it uses, derived here from the paper's forward equations:

* ``entmax_vjp`` -- Eq. 2: p_c = [(alpha-1) z_c - tau]_+^(1/(alpha-1)) with sum_c p_c = 1.  On the support
  dp_c = s_c (dz_c - dtau/(alpha-1)) with s_c = p_c^(2-alpha); summing over c and using sum dp = 0 gives
  dtau/(alpha-1) = sum_c s_c dz_c / sum_c s_c, hence J = diag(s) - s s^T / sum(s) on the support and 0 elsewhere.
* ``route_row_vjp`` -- Section 3.2 / Algorithm 2 / Proposition 1: z_hc = gamma <q_h, kbar_c>/sqrt(d), p_h = entmax(z_h),
  w_c = mean_h p_hc, bias_c = (log w_c - mean_{c' in S} log w_c')/sigma on the support S.
* ``attend_row_vjp`` -- Eq. 7 in the bias form of Proposition 1: logits l_j = <q, k_j>/sqrt(d) + bias_c(j) on routed
  tokens, + 0 on the diagonal tokens; P = softmax(l); o = P V.  With dP_j = <do, v_j> and delta = <o, do>:
  dl_j = P_j (dP_j - delta); dq = sum_j dl_j k_j / sqrt(d); dk_j = dl_j q / sqrt(d); dv_j = P_j do;
  dbias_c = sum over the heads of the group and the tokens of chunk c of dl_j.
* ``block_summaries_vjp`` -- Eq. 3: kbar_c = sum_t a_t k_t, a = softmax(<qbar, k_t>/sqrt(d)) over the chunk's tokens.

The support is piecewise constant in the inputs, so these are the gradients wherever no chunk sits exactly on the
threshold (the paper: "piecewise differentiable, analogous to sparsemax or ReLU").

``backward_prefill(..., through_routing=False)`` holds the routing (support and bias) fixed: the gradient of Stage 2
alone, which is what a Stage-2 backward kernel that is handed the mask and the bias lists computes (it also returns
dbias, the quantity such a kernel hands on to the routing backward).  ``through_routing=True`` is the whole method.

Pins (tests/test_oracle_backward.py): central finite differences of the forward oracle on tiny inputs (whole method,
every input including the summary query); the Jacobian against finite differences of ``entmax``, against the explicit
matrix, against the sparsemax (alpha = 2) and softmax (alpha -> 1) Jacobians; the fixed-routing gradient against
automatic differentiation of dense masked attention with an additive bias; sigma -> infinity makes the two agree.
"""
from __future__ import annotations

import math

import numpy as np

from . import dash_oracle as fwd

__all__ = ["entmax_vjp", "entmax_jacobian", "route_row_vjp", "attend_row_vjp", "block_summaries_vjp", "backward_prefill"]


def entmax_vjp(p: np.ndarray, dp: np.ndarray, alpha: float) -> np.ndarray:
    """dz = J^T dp for p = alpha-entmax(z) (z the unscaled scores of Eq. 2); J = diag(s) - s s^T / sum(s) is symmetric."""
    p = np.asarray(p, dtype=np.float64)
    dp = np.asarray(dp, dtype=np.float64)
    sup = p > 0.0
    s = np.zeros_like(p)
    s[sup] = p[sup] ** (2.0 - alpha)
    return s * (dp - float(s @ dp) / float(s.sum()))


def entmax_jacobian(p: np.ndarray, alpha: float) -> np.ndarray:
    """The matrix dp/dz at a point with output p (zero rows and columns outside the support)."""
    p = np.asarray(p, dtype=np.float64)
    s = np.where(p > 0.0, np.where(p > 0.0, p, 1.0) ** (2.0 - alpha), 0.0)
    return np.diag(s) - np.outer(s, s) / s.sum()


def route_row_vjp(q_g: np.ndarray, Kbar_r: np.ndarray, rt: fwd.RowRouting, dbias: np.ndarray, alpha: float,
                  gamma: float, sigma: float):
    """Backward of ``dash_oracle.route_row`` for the bias it outputs: (dq_g [g_q, d], dKbar [n_cand, d]).

    ``dbias`` [|S|] is the gradient w.r.t. the bias of each routed chunk (in the order of ``rt.support``).
    """
    q_g = np.asarray(q_g, dtype=np.float64)
    g_q, d = q_g.shape
    n_cand = rt.n_cand
    dq = np.zeros_like(q_g)
    dKbar = np.zeros((n_cand, d))
    S = rt.support
    if n_cand == 0 or S.size == 0:
        return dq, dKbar
    Kb = np.asarray(Kbar_r[:n_cand], dtype=np.float64)
    e = 1.0 / (alpha - 1.0)
    # bias_c = (log w_c - mu)/sigma, mu = mean over S of log w
    dlogw = (np.asarray(dbias, dtype=np.float64) - np.mean(dbias)) / sigma          # [|S|]
    dw = np.zeros(n_cand)
    dw[S] = dlogw / rt.w[S]
    # w_c = mean_h p_hc;  p_h = entmax_alpha(z_h) with z_h = x_h / (alpha - 1) = gamma <q_h, kbar>/sqrt(d)
    p = np.maximum(rt.x - rt.tau[:, None], 0.0) ** e                                  # [g_q, n_cand]
    scale = gamma / math.sqrt(d)
    for h in range(g_q):
        dz = entmax_vjp(p[h], dw / g_q, alpha)                                        # [n_cand]
        dq[h] = scale * (dz @ Kb)
        dKbar += scale * np.outer(dz, q_g[h])
    return dq, dKbar


def attend_row_vjp(q_g: np.ndarray, K_r: np.ndarray, V_r: np.ndarray, B: int, support: np.ndarray, bias: np.ndarray,
                   diag_lo: int, diag_hi: int, do_g: np.ndarray):
    """Backward of ``dash_oracle.attend_row``.  Returns (dq_g [g_q, d], tok [T] token ids, dk [T, d], dv [T, d],
    dbias [|S|]); the K / V gradients are those of the attended tokens ``tok`` only (every other token gets none)."""
    q_g = np.asarray(q_g, dtype=np.float64)
    do_g = np.asarray(do_g, dtype=np.float64)
    g_q, d = q_g.shape
    support = np.asarray(support, dtype=np.int64)
    routed, diag = fwd._attended_tokens(support, B, diag_lo, diag_hi)
    tok = np.concatenate([routed, diag])
    if tok.size == 0:
        return np.zeros_like(q_g), tok, np.zeros((0, d)), np.zeros((0, d)), np.zeros(0)
    Kt = np.asarray(K_r, dtype=np.float64)[tok]
    Vt = np.asarray(V_r, dtype=np.float64)[tok]
    dj = np.concatenate([np.repeat(np.asarray(bias, dtype=np.float64), B), np.zeros(diag.size)])
    logits = q_g @ Kt.T / math.sqrt(d) + dj[None, :]
    logits = logits - logits.max(axis=1, keepdims=True)
    P = np.exp(logits)
    P = P / P.sum(axis=1, keepdims=True)                     # [g_q, T]
    o = P @ Vt
    dP = do_g @ Vt.T                                         # [g_q, T]
    delta = np.sum(o * do_g, axis=1, keepdims=True)          # [g_q, 1]
    dl = P * (dP - delta)                                    # [g_q, T]
    dq = dl @ Kt / math.sqrt(d)
    dk = dl.T @ q_g / math.sqrt(d)
    dv = P.T @ do_g
    dbias = dl[:, :routed.size].sum(axis=0).reshape(support.size, B).sum(axis=1) if support.size else np.zeros(0)
    return dq, tok, dk, dv, dbias


def block_summaries_vjp(K: np.ndarray, B: int, qbar, dKbar: np.ndarray):
    """Backward of ``dash_oracle.block_summaries`` for one sequence: K [n, h_kv, d], dKbar [T_s, h_kv, d].

    Returns (dK [n, h_kv, d], dqbar of qbar's shape or None).
    """
    K = np.asarray(K, dtype=np.float64)
    n, h_kv, d = K.shape
    T_s = dKbar.shape[0]
    dK = np.zeros_like(K)
    dqbar = None if qbar is None else np.zeros_like(np.asarray(qbar, dtype=np.float64))
    for c in range(T_s):
        for r in range(h_kv):
            Kc = K[c * B:(c + 1) * B, r, :]
            g = dKbar[c, r]
            if qbar is None:
                dK[c * B:(c + 1) * B, r, :] += g[None, :] / B
                continue
            qb = np.asarray(qbar, dtype=np.float64)
            qv = qb[r] if qb.ndim == 2 else qb[c, r]
            s = Kc @ qv / math.sqrt(d)
            s = s - s.max()
            a = np.exp(s)
            a = a / a.sum()
            da = Kc @ g                                      # d kbar / d a_t = k_t
            ds = a * (da - float(a @ da))
            dK[c * B:(c + 1) * B, r, :] += a[:, None] * g[None, :] + np.outer(ds, qv) / math.sqrt(d)
            dq = ds @ Kc / math.sqrt(d)
            if qb.ndim == 2:
                dqbar[r] += dq
            else:
                dqbar[c, r] += dq
    return dK, dqbar


def backward_prefill(Q: np.ndarray, K: np.ndarray, V: np.ndarray, dO: np.ndarray, *, B: int, alpha: float,
                     gamma: float = 1.0, sigma: float = 10.0, qbar=None, local_blocks: int = 0,
                     through_routing: bool = True, rows=None, kv_heads=None):
    """Gradients of L = sum(O * dO) for a causal prefill over [b, n, h, d] tensors (plain loops: small inputs only).

    Returns dict(dQ, dK, dV [like the inputs], dqbar or None, dbias {(b, r, i): [|S_i|]}).  With
    ``through_routing=False`` the routing is held fixed (no gradient into Stage 1 / Stage 0).  ``rows`` / ``kv_heads``
    restrict the rows whose loss terms are included (dK / dV then hold only their contributions).
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    b, n, h_q, d = Q.shape
    h_kv = K.shape[2]
    g_q = h_q // h_kv
    dQ, dK, dV = np.zeros_like(Q), np.zeros_like(K), np.zeros_like(V)
    dqbar = None if qbar is None else np.zeros_like(np.asarray(qbar, dtype=np.float64))
    dbias_all = {}
    rows = range(n) if rows is None else rows
    kv_heads = range(h_kv) if kv_heads is None else kv_heads
    for bb in range(b):
        Kbar = fwd.block_summaries(K[bb], B, qbar)
        dKbar = np.zeros_like(Kbar)
        for r in kv_heads:
            for i in rows:
                q_g = Q[bb, i, r * g_q:(r + 1) * g_q]
                n_cand, dlo, dhi = fwd._row_geometry(i, n, B, True, local_blocks)
                rt = fwd.route_row(q_g, Kbar[:, r, :], n_cand, alpha, gamma, sigma)
                dq, tok, dk, dv, dbias = attend_row_vjp(q_g, K[bb, :, r, :], V[bb, :, r, :], B, rt.support, rt.bias, dlo,
                                                        dhi, dO[bb, i, r * g_q:(r + 1) * g_q])
                dQ[bb, i, r * g_q:(r + 1) * g_q] += dq
                np.add.at(dK[bb, :, r, :], tok, dk)
                np.add.at(dV[bb, :, r, :], tok, dv)
                dbias_all[(bb, r, i)] = dbias
                if through_routing and rt.support.size:
                    dq2, dkb = route_row_vjp(q_g, Kbar[:, r, :], rt, dbias, alpha, gamma, sigma)
                    dQ[bb, i, r * g_q:(r + 1) * g_q] += dq2
                    dKbar[:n_cand, r, :] += dkb
        if through_routing:
            dK0, dqb = block_summaries_vjp(K[bb], B, qbar, dKbar)
            dK[bb] += dK0
            if dqb is not None:
                dqbar += dqb
    return {"dQ": dQ, "dK": dK, "dV": dV, "dqbar": dqbar, "dbias": dbias_all}
