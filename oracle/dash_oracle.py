"""Float64 CPU oracle for the DashAttention forward pass.

TEST INFRASTRUCTURE ONLY.  This module is the plain, slow, by-the-definition
statement of what the forward pass computes.  It shares no code with the CUDA
path and nothing in the product package imports it; only the tests, the smoke
check and the benchmark's CPU-baseline leg call it.

Everything is numpy float64.  Index convention: 0-based token positions
``i, j in [0, n)``; chunk of token ``j`` is ``j // B``; ``c_i = i // B`` is the
query's own ("diagonal") chunk; only *complete* chunks have summaries
(Algorithm 1, step 1: T_c = floor(n / B)).

Passages followed (paper's numbering):

* Eq. 2 / appendix "The alpha-entmax mapping": ``entmax_threshold``, ``entmax``.
* Eq. 3 / Algorithm 1: ``block_summaries``.
* Section 3.2 (chunk logits, Eq. 4, GQA averaging) / Algorithm 2: ``route_row``.
* Proposition 1 / Algorithm 2 second pass: the bias inside ``route_row``.
* Eq. 7 in the bias form of Proposition 1 / Algorithm 3: ``attend_row``.
* Eq. 6, 8, 9, 10 (the definition form): ``attend_row_definition_form``.

Readings where the paper is silent or inconsistent (each also listed in the
design notes):

* gamma (also written t_c in the paper's appendix) multiplies the chunk logit.
* Routed candidates of row i are the chunks strictly before c_i (Algorithm 2,
  the sum over c < c_i); the diagonal chunk is never scored and always attended
  with bias 0 and a causal mask (Algorithm 2 last step, Algorithm 3 step 7).
* |R_i| and |D_i| in Eq. 9-10 count tokens (the proof of Proposition 1 does).
* Support test: a chunk is routed iff its largest per-head margin
  ``x - tau`` is > 0.  Equal to ``w > 0`` in exact arithmetic, immune to
  underflow of ``margin ** (1/(alpha-1))``.
* log w is evaluated in a scaled form so that tiny weights do not underflow.
* Rows of chunk 0 have no candidate: Stage 1 is skipped, the output is the
  causal softmax inside chunk 0.
* Non-causal mode (the paper is causal throughout): candidates are all complete
  chunks; D_i is the incomplete tail chunk (empty when B divides n), bias 0.
  Parity unpinned by the paper beyond brute force on tiny inputs.
* Decode: ``kv_len`` counts the new token; the query sits at ``kv_len - 1``.
* Local window (``local_blocks = L``; appendix "Long-context adaptation", training
  settings: the sliding window is the diagonal block and the last block).  Read
  as: the L chunks just before the diagonal chunk belong to D_i together with
  the causal part of the diagonal chunk: attended in full with bias 0, counted
  in |D_i|, and not scored, so the routed candidates are the chunks before
  c_i - L.  L = 0 is Algorithms 2-3 as printed; L = 1 with B = 64 gives
  |D_i| = 64 + (i mod 64) + 1 tokens (the appendix counts "64-127", i.e.
  without the query's own position).  The other possible reading (the previous
  chunk forced into the support but still scored) is not built; parity between
  the two is unpinned by the paper.  Causal mode only.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

__all__ = [
    "entmax_threshold", "entmax_threshold_bisect", "entmax",
    "block_summaries", "route_row", "attend_row", "attend_row_definition_form",
    "RowRouting", "forward_row", "forward_prefill", "forward_decode",
    "pack_mask_words", "block_sparsity", "selected_flops",
]


# --------------------------------------------------------------------------
# Eq. 2: alpha-entmax.  Throughout, ``x`` is the already scaled score
# (alpha - 1) * s, so the output is [x - tau]_+ ** (1 / (alpha - 1)).
# --------------------------------------------------------------------------

def _check_alpha(alpha: float) -> float:
    alpha = float(alpha)
    if not alpha > 1.0:
        raise ValueError("alpha must be > 1 (alpha -> 1 is softmax, handled by the caller)")
    return alpha


def entmax_threshold_bisect(x: np.ndarray, alpha: float) -> float:
    """Root tau of f(tau) = sum_c [x_c - tau]_+^(1/(alpha-1)) - 1 (Eq. 2), any alpha > 1.

    f is continuous and strictly decreasing on (-inf, max x).  At
    tau = max x - 1 the largest term alone is 1, so f >= 0; at
    tau = max x - k^(-(alpha-1)) every one of the k terms is at most 1/k, so
    f <= 0.  Bisect that bracket until it no longer shrinks in float64, then
    take Newton steps on the support found (f is smooth there).
    """
    alpha = _check_alpha(alpha)
    x = np.asarray(x, dtype=np.float64).ravel()
    if x.size == 0:
        raise ValueError("entmax of an empty vector is undefined")
    e = 1.0 / (alpha - 1.0)
    xmax = float(x.max())
    lo = xmax - 1.0
    hi = xmax - float(x.size) ** (-(alpha - 1.0))

    def f(t: float) -> float:
        return float(np.sum(np.maximum(x - t, 0.0) ** e)) - 1.0

    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if mid <= lo or mid >= hi:
            break
        if f(mid) >= 0.0:
            lo = mid
        else:
            hi = mid
    tau = lo
    # Newton polish on the fixed support {x > tau}; f'(tau) = -e * sum m^(e-1).
    for _ in range(8):
        m = x[x > tau] - tau
        if m.size == 0:
            break
        g = float(np.sum(m ** e)) - 1.0
        dg = -e * float(np.sum(m ** (e - 1.0)))
        if dg == 0.0:
            break
        new = tau - g / dg
        if not (xmax - 1.0 <= new < xmax):
            break
        if new == tau:
            break
        tau = new
    return float(tau)


def _threshold_alpha2_sorted(x: np.ndarray) -> float:
    """alpha = 2 (sparsemax): sort descending, k* = max{k : x_(k) > (sum_{<=k} x - 1)/k}."""
    xs = np.sort(x)[::-1]
    cs = np.cumsum(xs)
    k = np.arange(1, xs.size + 1, dtype=np.float64)
    tau_k = (cs - 1.0) / k
    kstar = int(np.nonzero(xs > tau_k)[0].max())
    return float(tau_k[kstar])


def _threshold_alpha15_sorted(x: np.ndarray) -> float:
    """alpha = 1.5: sum_{<=k} (x - tau)^2 = ss_k + k (mean_k - tau)^2 = 1 on the top-k prefix."""
    xs = np.sort(x)[::-1]
    k = np.arange(1, xs.size + 1, dtype=np.float64)
    mean = np.cumsum(xs) / k
    # ss_k = sum_{<=k} (x - mean_k)^2, from the two running sums
    ss = np.cumsum(xs * xs) - k * mean * mean
    # the difference of two large sums can be slightly negative; it is a sum of squares
    ss = np.maximum(ss, 0.0)
    delta = np.maximum((1.0 - ss) / k, 0.0)
    tau_k = mean - np.sqrt(delta)
    kstar = int(np.nonzero(xs > tau_k)[0].max())
    # re-evaluate on the chosen prefix with a two-pass variance (no cancellation)
    top = xs[:kstar + 1]
    m = float(top.mean())
    ssk = float(((top - m) ** 2).sum())
    return m - math.sqrt(max((1.0 - ssk) / top.size, 0.0))


def entmax_threshold(x: np.ndarray, alpha: float) -> float:
    """The unique tau of Eq. 2 for scaled scores ``x``.

    alpha = 2 and alpha = 1.5 use the exact sort-based procedures; every other
    alpha uses bisection + Newton.  For the two special cases the sort is run
    on scores shifted by their maximum (entmax is shift invariant), which
    keeps the running sums of squares well conditioned.
    """
    alpha = _check_alpha(alpha)
    x = np.asarray(x, dtype=np.float64).ravel()
    if x.size == 0:
        raise ValueError("entmax of an empty vector is undefined")
    xmax = float(x.max())
    if alpha == 2.0:
        return _threshold_alpha2_sorted(x - xmax) + xmax
    if alpha == 1.5:
        return _threshold_alpha15_sorted(x - xmax) + xmax
    return entmax_threshold_bisect(x, alpha)


def entmax(s: np.ndarray, alpha: float) -> np.ndarray:
    """alpha-entmax of raw scores ``s`` (Eq. 2): [(alpha-1) s - tau]_+^(1/(alpha-1))."""
    alpha = _check_alpha(alpha)
    s = np.asarray(s, dtype=np.float64)
    x = (alpha - 1.0) * s.ravel()
    tau = entmax_threshold(x, alpha)
    return (np.maximum(x - tau, 0.0) ** (1.0 / (alpha - 1.0))).reshape(s.shape)


# --------------------------------------------------------------------------
# Eq. 3 / Algorithm 1: chunk summaries.
# --------------------------------------------------------------------------

def block_summaries(K: np.ndarray, B: int, qbar: np.ndarray | None = None,
                    kv_len: int | None = None) -> np.ndarray:
    """Summaries of the complete chunks of one sequence.

    K: [n, h_kv, d].  qbar: None (zero summary query: mean pooling), [h_kv, d]
    (one query per head) or [T, h_kv, d] (one per chunk and head).
    Returns Kbar [T_s, h_kv, d] with T_s = floor(len / B), len = kv_len or n.
    """
    K = np.asarray(K, dtype=np.float64)
    n, h_kv, d = K.shape
    length = n if kv_len is None else int(kv_len)
    T_s = length // B
    out = np.zeros((T_s, h_kv, d), dtype=np.float64)
    for c in range(T_s):
        for r in range(h_kv):
            Kc = K[c * B:(c + 1) * B, r, :]                      # [B, d]
            if qbar is None:
                a = np.full(B, 1.0 / B)
            else:
                qb = np.asarray(qbar, dtype=np.float64)
                qv = qb[r] if qb.ndim == 2 else qb[c, r]
                s = Kc @ qv / math.sqrt(d)
                s = s - s.max()
                a = np.exp(s)
                a = a / a.sum()
            out[c, r, :] = a @ Kc
    return out


# --------------------------------------------------------------------------
# Stage 1 for one (row, KV head): Algorithm 2 + Proposition 1.
# --------------------------------------------------------------------------

@dataclass
class RowRouting:
    """Stage-1 result of one query row and one KV head."""
    n_cand: int                                   # number of candidate chunks
    x: np.ndarray = field(default_factory=lambda: np.zeros((0, 0)))       # [g_q, n_cand] scaled logits
    tau: np.ndarray = field(default_factory=lambda: np.zeros(0))          # [g_q]
    margin: np.ndarray = field(default_factory=lambda: np.zeros(0))       # [n_cand] max_h (x - tau)
    w: np.ndarray = field(default_factory=lambda: np.zeros(0))            # [n_cand] group weights
    support: np.ndarray = field(default_factory=lambda: np.zeros(0, dtype=np.int64))  # routed chunk ids, ascending
    bias: np.ndarray = field(default_factory=lambda: np.zeros(0))         # [len(support)] d of Prop. 1
    log_w: np.ndarray = field(default_factory=lambda: np.zeros(0))        # [len(support)]
    local: np.ndarray = field(default_factory=lambda: np.zeros(0, dtype=np.int64))  # window chunks before the diagonal one


def route_row(q_g: np.ndarray, Kbar_r: np.ndarray, n_cand: int, alpha: float,
              gamma: float, sigma: float) -> RowRouting:
    """Route one row.  q_g: [g_q, d] query heads of the group; Kbar_r: [>= n_cand, d].

    x = gamma (alpha-1) <q, kbar> / sqrt(d)      (Algorithm 2, step 1)
    tau_h: root of sum_c [x_hc - tau]_+^(1/(alpha-1)) = 1 per head (step 5)
    w_c = mean_h [x_hc - tau_h]_+^(1/(alpha-1))  (step 9, Section 3.2)
    support = {c : max_h (x_hc - tau_h) > 0}     (step 10, union of head supports)
    mu = mean_{c in support} log w_c; d_c = (log w_c - mu) / sigma (Prop. 1)
    """
    alpha = _check_alpha(alpha)
    q_g = np.asarray(q_g, dtype=np.float64)
    g_q, d = q_g.shape
    if n_cand <= 0:
        return RowRouting(n_cand=0)
    e = 1.0 / (alpha - 1.0)
    x = gamma * (alpha - 1.0) * (q_g @ np.asarray(Kbar_r[:n_cand], dtype=np.float64).T) / math.sqrt(d)
    tau = np.array([entmax_threshold(x[h], alpha) for h in range(g_q)])
    marg = x - tau[:, None]                                   # [g_q, n_cand]
    margin = marg.max(axis=0)
    support = np.nonzero(margin > 0.0)[0]
    pos = np.maximum(marg, 0.0)
    w = (pos ** e).mean(axis=0)
    # log w_c = e log m* + log sum_h (m_h / m*)^e - log g_q with m* the largest positive margin
    ms = pos[:, support]                                      # [g_q, |S|]
    mstar = ms.max(axis=0)
    log_w = e * np.log(mstar) + np.log(((ms / mstar) ** e).sum(axis=0)) - math.log(g_q)
    mu = log_w.mean()
    bias = (log_w - mu) / sigma
    return RowRouting(n_cand=n_cand, x=x, tau=tau, margin=margin, w=w,
                      support=support.astype(np.int64), bias=bias, log_w=log_w)


# --------------------------------------------------------------------------
# Stage 2 for one (row, KV head).
# --------------------------------------------------------------------------

def _attended_tokens(support: np.ndarray, B: int, diag_lo: int, diag_hi: int):
    """Token ids of the routed chunks followed by the diagonal tokens [diag_lo, diag_hi)."""
    routed = (support[:, None] * B + np.arange(B)[None, :]).ravel() if support.size else np.zeros(0, dtype=np.int64)
    diag = np.arange(diag_lo, diag_hi, dtype=np.int64)
    return routed.astype(np.int64), diag


def attend_row(q_g: np.ndarray, K_r: np.ndarray, V_r: np.ndarray, B: int,
               support: np.ndarray, bias: np.ndarray, diag_lo: int, diag_hi: int) -> np.ndarray:
    """Eq. 7 in the bias form of Proposition 1, one-shot softmax.

    q_g [g_q, d]; K_r, V_r [len, d]; routed chunks ``support`` with per-chunk
    bias; diagonal tokens [diag_lo, diag_hi) with bias 0.  Returns [g_q, d].
    """
    q_g = np.asarray(q_g, dtype=np.float64)
    d = q_g.shape[1]
    routed, diag = _attended_tokens(np.asarray(support, dtype=np.int64), B, diag_lo, diag_hi)
    tok = np.concatenate([routed, diag])
    if tok.size == 0:
        return np.zeros_like(q_g)
    dj = np.concatenate([np.repeat(np.asarray(bias, dtype=np.float64), B), np.zeros(diag.size)])
    logits = q_g @ np.asarray(K_r, dtype=np.float64)[tok].T / math.sqrt(d) + dj[None, :]
    logits = logits - logits.max(axis=1, keepdims=True)
    p = np.exp(logits)
    p = p / p.sum(axis=1, keepdims=True)
    return p @ np.asarray(V_r, dtype=np.float64)[tok]


def attend_row_definition_form(q_g: np.ndarray, K_r: np.ndarray, V_r: np.ndarray, B: int,
                               support: np.ndarray, w_support: np.ndarray, sigma: float,
                               diag_lo: int, diag_hi: int) -> np.ndarray:
    """Eq. 6 with the prior g_sigma(w) built from Eq. 8, 9 and 10 (no bias shortcut).

    w'_j = (1/B) w_c(j)^(1/sigma) / sum_c w_c^(1/sigma)                       (Eq. 8)
    lambda = sigmoid(KL(u_R || w'_R) + log(|R| / |D|)), |R|, |D| in tokens    (Eq. 10)
    g_j = lambda w'_j on R, (1 - lambda)/|D| on D                             (Eq. 9)
    p_j = g_j exp(z_j) / sum_t g_t exp(z_t)                                   (Eq. 6)
    """
    q_g = np.asarray(q_g, dtype=np.float64)
    d = q_g.shape[1]
    support = np.asarray(support, dtype=np.int64)
    routed, diag = _attended_tokens(support, B, diag_lo, diag_hi)
    nR, nD = routed.size, diag.size
    if nR + nD == 0:
        return np.zeros_like(q_g)
    if nR == 0:
        g = np.full(nD, 1.0 / nD)
    else:
        ws = np.asarray(w_support, dtype=np.float64) ** (1.0 / sigma)
        wprime = np.repeat(ws / (B * ws.sum()), B)                        # per routed token
        if nD == 0:
            g = wprime                                                     # all mass on R
        else:
            kl = float(np.sum((1.0 / nR) * np.log((1.0 / nR) / wprime)))
            a = kl + math.log(nR / nD)
            lam = 1.0 / (1.0 + math.exp(-a))
            g = np.concatenate([lam * wprime, np.full(nD, (1.0 - lam) / nD)])
    tok = np.concatenate([routed, diag])
    z = q_g @ np.asarray(K_r, dtype=np.float64)[tok].T / math.sqrt(d)
    z = z - z.max(axis=1, keepdims=True)
    num = g[None, :] * np.exp(z)
    p = num / num.sum(axis=1, keepdims=True)
    return p @ np.asarray(V_r, dtype=np.float64)[tok]


# --------------------------------------------------------------------------
# Whole rows / whole problems.
# --------------------------------------------------------------------------

def _row_geometry(i: int, length: int, B: int, causal: bool, local_blocks: int = 0):
    """(number of candidate chunks, token range of D_i) of query position i.

    With a local window of L chunks, D_i starts L chunks before the diagonal
    chunk (or at token 0) and the candidates are the chunks before that.
    """
    T_s = length // B
    if local_blocks < 0:
        raise ValueError("local_blocks must be >= 0")
    if causal:
        c_lo = max(i // B - local_blocks, 0)
        return min(c_lo, T_s), c_lo * B, i + 1
    if local_blocks:
        raise ValueError("the local window is defined for the causal mode only")
    return T_s, T_s * B, length


def forward_row(Q_b: np.ndarray, K_b: np.ndarray, V_b: np.ndarray, Kbar_b: np.ndarray,
                i: int, r: int, *, B: int, alpha: float, gamma: float, sigma: float,
                causal: bool = True, length: int | None = None, q_row: np.ndarray | None = None,
                local_blocks: int = 0):
    """One query row i of KV head r of one sequence.

    Q_b [n, h_q, d] (or pass ``q_row`` [h_q, d] for decode), K_b, V_b
    [>= length, h_kv, d], Kbar_b [T_s, h_kv, d].  Returns (RowRouting, O [g_q, d]).
    """
    h_kv = K_b.shape[1]
    qh = Q_b[i] if q_row is None else q_row                     # [h_q, d]
    g_q = qh.shape[0] // h_kv
    q_g = np.asarray(qh[r * g_q:(r + 1) * g_q], dtype=np.float64)
    length = K_b.shape[0] if length is None else int(length)
    n_cand, dlo, dhi = _row_geometry(i, length, B, causal, local_blocks)
    rt = route_row(q_g, Kbar_b[:, r, :], n_cand, alpha, gamma, sigma)
    if causal:
        rt.local = np.arange(dlo // B, i // B, dtype=np.int64)
    o = attend_row(q_g, K_b[:length, r, :], V_b[:length, r, :], B, rt.support, rt.bias, dlo, dhi)
    return rt, o


def pack_mask_words(support: np.ndarray, diag_chunk: int | None, n_words: int) -> np.ndarray:
    """Bit-pack a row's routed chunks (+ the diagonal chunk) LSB-first: chunk c -> bit c%32 of word c//32."""
    words = np.zeros(n_words, dtype=np.uint32)
    ids = list(np.asarray(support, dtype=np.int64))
    if diag_chunk is not None:
        ids.append(int(diag_chunk))
    for c in ids:
        words[c >> 5] |= np.uint32(1) << np.uint32(c & 31)
    return words


def forward_prefill(Q: np.ndarray, K: np.ndarray, V: np.ndarray, *, B: int, alpha: float,
                    gamma: float = 1.0, sigma: float = 10.0, causal: bool = True,
                    qbar: np.ndarray | None = None, rows=None, kv_heads=None, local_blocks: int = 0):
    """Prefill over [b, n, h, d] tensors.  ``rows``/``kv_heads`` restrict the work to a sample.

    Returns a dict: Kbar [b, T_s, h_kv, d]; O [b, n, h_q, d] (NaN where not
    computed); routing[(b, r, i)] -> RowRouting.
    """
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    b, n, h_q, d = Q.shape
    h_kv = K.shape[2]
    g_q = h_q // h_kv
    rows = range(n) if rows is None else rows
    kv_heads = range(h_kv) if kv_heads is None else kv_heads
    O = np.full((b, n, h_q, d), np.nan)
    Kbar = np.stack([block_summaries(K[bb], B, qbar) for bb in range(b)])
    routing = {}
    for bb in range(b):
        for r in kv_heads:
            for i in rows:
                rt, o = forward_row(Q[bb], K[bb], V[bb], Kbar[bb], i, r, B=B, alpha=alpha,
                                    gamma=gamma, sigma=sigma, causal=causal, local_blocks=local_blocks)
                routing[(bb, r, i)] = rt
                O[bb, i, r * g_q:(r + 1) * g_q, :] = o
    return {"Kbar": Kbar, "O": O, "routing": routing}


def forward_decode(Q: np.ndarray, Kc: np.ndarray, Vc: np.ndarray, kv_len, *, B: int, alpha: float,
                   gamma: float = 1.0, sigma: float = 10.0, qbar: np.ndarray | None = None,
                   Kbar: np.ndarray | None = None, batches=None, kv_heads=None, local_blocks: int = 0):
    """Decode: Q [b, h_q, d] (one new token per sequence), caches [b, cap, h_kv, d], kv_len [b].

    The query of sequence bb sits at position kv_len[bb] - 1 (the new token is
    already in the cache).  Equals the last row of a causal prefill of that length.
    """
    Q = np.asarray(Q, dtype=np.float64)
    b, h_q, d = Q.shape
    h_kv = Kc.shape[2]
    g_q = h_q // h_kv
    O = np.full((b, h_q, d), np.nan)
    routing = {}
    batches = range(b) if batches is None else batches
    kv_heads = range(h_kv) if kv_heads is None else kv_heads
    for bb in batches:
        L = int(kv_len[bb])
        if Kbar is None:
            Kb = None
        else:
            Kb = np.asarray(Kbar[bb], dtype=np.float64)
        for r in kv_heads:
            K_b = np.asarray(Kc[bb, :L, r:r + 1, :], dtype=np.float64)
            V_b = np.asarray(Vc[bb, :L, r:r + 1, :], dtype=np.float64)
            if Kb is None:
                qb = None
                if qbar is not None:
                    qa = np.asarray(qbar, dtype=np.float64)
                    qb = qa[r:r + 1] if qa.ndim == 2 else qa[:, r:r + 1]
                Kbar_r = block_summaries(K_b, B, qb)
            else:
                Kbar_r = Kb[:, r:r + 1, :]
            q_row = Q[bb, r * g_q:(r + 1) * g_q, :]
            rt, o = forward_row(None, K_b, V_b, Kbar_r, L - 1, 0, B=B, alpha=alpha, gamma=gamma,
                                sigma=sigma, causal=True, length=L, q_row=q_row, local_blocks=local_blocks)
            routing[(bb, r)] = rt
            O[bb, r * g_q:(r + 1) * g_q, :] = o
    return {"O": O, "routing": routing}


# --------------------------------------------------------------------------
# Workload statistics (definitions used by the reports).
# --------------------------------------------------------------------------

def block_sparsity(support_sizes: np.ndarray, visible_chunks: np.ndarray) -> float:
    """1 - sum(|S_i| + 1) / sum(c_i + 1): fraction of visible chunks not attended (diagonal on both sides)."""
    s = np.asarray(support_sizes, dtype=np.float64)
    v = np.asarray(visible_chunks, dtype=np.float64)
    return float(1.0 - (s + 1.0).sum() / (v + 1.0).sum())


def selected_flops(support_sizes: np.ndarray, diag_tokens: np.ndarray, B: int, d: int, g_q: int) -> float:
    """4 d g_q sum_rows (B |S_i| + |D_i|): QK^T and PV multiply-adds over attended tokens only."""
    s = np.asarray(support_sizes, dtype=np.float64)
    dt = np.asarray(diag_tokens, dtype=np.float64)
    return float(4.0 * d * g_q * (B * s + dt).sum())
