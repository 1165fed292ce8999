"""Pins for the oracle's Stage 0 / 1 / 2 against what the paper fixes: mean pooling at a zero
summary query, simplex invariants of the routing weights, Proposition 1 (bias form ==
definition form), the closed form of lambda, the sigma -> infinity limit, brute-force dense
masked attention through an independent library routine, and decode == last prefill row."""
import math

import numpy as np
import pytest
import torch

from oracle import dash_oracle as orc


def _rand(shape, seed, scale=1.0):
    return np.random.default_rng(seed).normal(size=shape) * scale


# ----------------------------------------------------------------- Stage 0 (Eq. 3)

def test_zero_summary_query_is_mean_pooling():
    K = _rand((200, 3, 16), 0)
    kb = orc.block_summaries(K, 64, qbar=np.zeros((3, 16)))
    assert kb.shape == (3, 3, 16)          # only complete chunks
    assert np.allclose(kb, K[:192].reshape(3, 64, 3, 16).mean(axis=1), atol=1e-14)
    assert np.allclose(orc.block_summaries(K, 64, qbar=None), kb, atol=1e-14)


def test_summary_is_local_softmax_average():
    """Eq. 3 as torch's library attention: one query (qbar) attending inside one chunk."""
    K = _rand((128, 2, 8), 1)
    qbar = _rand((2, 8), 2, 2.0)
    kb = orc.block_summaries(K, 32, qbar)
    Kt = torch.from_numpy(K)
    for c in range(4):
        for r in range(2):
            kc = Kt[c * 32:(c + 1) * 32, r][None]
            ref = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(qbar[r])[None, None], kc, kc)[0, 0].numpy()
            assert np.allclose(kb[c, r], ref, atol=1e-13)


def test_summary_depends_only_on_own_chunk_and_per_chunk_queries():
    K = _rand((256, 1, 8), 3)
    qb = _rand((4, 1, 8), 4)
    full = orc.block_summaries(K, 64, qb)
    K2 = K.copy()
    K2[64:128] += 5.0
    other = orc.block_summaries(K2, 64, qb)
    assert np.array_equal(full[[0, 2, 3]], other[[0, 2, 3]]) and not np.allclose(full[1], other[1])
    # prefix (incremental) computation gives the same summaries
    assert np.array_equal(orc.block_summaries(K, 64, qb, kv_len=130), full[:2])


# ----------------------------------------------------------------- Stage 1 (Algorithm 2)

@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
def test_group_weights_on_simplex_and_support_is_union(alpha):
    d, g_q, T = 16, 4, 40
    q = _rand((g_q, d), 5, 1.5)
    kbar = _rand((T, d), 6)
    rt = orc.route_row(q, kbar, T, alpha, gamma=2.0, sigma=10.0)
    assert abs(rt.w.sum() - 1.0) < 1e-12 and np.all(rt.w >= 0)
    union = set()
    for h in range(g_q):
        s = 2.0 * (q[h] @ kbar.T) / math.sqrt(d)
        p = orc.entmax(s, alpha)                       # per-head entmax of gamma * zbar (Eq. 4)
        union |= set(np.nonzero(p > 0)[0])
        assert np.allclose(p, np.maximum(rt.x[h] - rt.tau[h], 0) ** (1 / (alpha - 1)), atol=1e-12)
    assert set(rt.support) == union == set(np.nonzero(rt.w > 0)[0])
    assert np.allclose(rt.log_w, np.log(rt.w[rt.support]), atol=1e-12)
    assert abs(rt.bias.mean()) < 1e-13                 # d sums to zero over the support
    assert np.allclose(rt.bias, (np.log(rt.w[rt.support]) - np.log(rt.w[rt.support]).mean()) / 10.0)


def test_gamma_sharpens_routing():
    q = _rand((2, 32), 7)
    kbar = _rand((100, 32), 8)
    sizes = [orc.route_row(q, kbar, 100, 1.5, g, 10.0).support.size for g in (0.25, 1.0, 4.0, 16.0)]
    assert sizes == sorted(sizes, reverse=True) and sizes[0] > sizes[-1]


def test_log_w_survives_underflow():
    """alpha = 1.25 raises the margin to the 4th power: margins near 1e-90 underflow w but not log w."""
    q = np.array([[1.0, 0.0]])
    kbar = np.array([[4.0, 0.0], [4.0 - 1e-60, 0.0], [0.0, 0.0]])
    rt = orc.route_row(q, kbar, 3, 1.25, 1.0, 1.0)
    assert np.all(np.isfinite(rt.log_w)) and np.all(np.isfinite(rt.bias))


# ----------------------------------------------------------------- Stage 2 (Eq. 6-10, Prop. 1)

def _case(seed, n=200, B=16, h_kv=2, g_q=2, d=8, scale=2.0):
    Q = _rand((1, n, h_kv * g_q, d), seed, scale)
    K = _rand((1, n, h_kv, d), seed + 1, scale)
    V = _rand((1, n, h_kv, d), seed + 2)
    return Q, K, V


@pytest.mark.parametrize("sigma", [1.0, 10.0, 1e4, 1e8])
@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
def test_proposition1_bias_form_equals_definition_form(alpha, sigma):
    Q, K, V = _case(20)
    B = 16
    Kbar = orc.block_summaries(K[0], B)
    for i in (0, 15, 16, 17, 63, 100, 199):
        for r in (0, 1):
            rt, o = orc.forward_row(Q[0], K[0], V[0], Kbar, i, r, B=B, alpha=alpha, gamma=3.0, sigma=sigma)
            c_i = i // B
            o2 = orc.attend_row_definition_form(Q[0, i, 2 * r:2 * r + 2], K[0, :, r], V[0, :, r], B,
                                                rt.support, rt.w[rt.support] if rt.n_cand else np.zeros(0),
                                                sigma, c_i * B, i + 1)
            assert np.allclose(o, o2, rtol=1e-11, atol=1e-12)


def test_prior_is_a_distribution_with_closed_form_lambda():
    """Eq. 9: g sums to 1 with mass lambda on R; proof of Prop. 1: lambda = 1/(1 + |D| eta),
    eta the geometric mean of w' over routed tokens; sigma -> inf: lambda -> |R|/(|R|+|D|)."""
    B = 8
    w = np.array([0.5, 0.3, 0.2])
    for sigma in (1.0, 3.0, 50.0, 1e9):
        ws = w ** (1 / sigma)
        wprime = np.repeat(ws / (B * ws.sum()), B)
        nR, nD = wprime.size, 5
        kl = np.sum((1 / nR) * np.log((1 / nR) / wprime))
        lam = 1 / (1 + math.exp(-(kl + math.log(nR / nD))))
        eta = np.exp(np.log(wprime).mean())
        assert abs(lam - 1 / (1 + nD * eta)) < 1e-13
        g = np.concatenate([lam * wprime, np.full(nD, (1 - lam) / nD)])
        assert abs(g.sum() - 1) < 1e-13 and abs(g[:nR].sum() - lam) < 1e-13
    assert abs(lam - nR / (nR + nD)) < 1e-8


def _dense_reference(Q, K, V, routing, B, h_kv, g_q):
    """Token-level additive mask (bias on routed tokens, 0 on the causal diagonal part, -inf elsewhere)
    fed to torch's scaled_dot_product_attention in float64 (Eq. 1 with M = bias/mask)."""
    n, d = Q.shape[1], Q.shape[3]
    out = np.zeros((n, h_kv * g_q, d))
    for r in range(h_kv):
        M = np.full((n, n), -np.inf)
        for i in range(n):
            rt = routing[(0, r, i)]
            for c, dc in zip(rt.support, rt.bias):
                M[i, c * B:(c + 1) * B] = dc
            M[i, (i // B) * B:i + 1] = 0.0
        for h in range(r * g_q, (r + 1) * g_q):
            o = torch.nn.functional.scaled_dot_product_attention(
                torch.from_numpy(Q[0, :, h])[None], torch.from_numpy(K[0, :, r])[None],
                torch.from_numpy(V[0, :, r])[None], attn_mask=torch.from_numpy(M)[None])
            out[:, h] = o[0].numpy()
    return out


@pytest.mark.parametrize("alpha,n", [(1.5, 200), (2.0, 131), (1.25, 64)])
def test_prefill_equals_dense_masked_attention(alpha, n):
    Q, K, V = _case(30, n=n)
    res = orc.forward_prefill(Q, K, V, B=16, alpha=alpha, gamma=3.0, sigma=2.0)
    ref = _dense_reference(Q, K, V, res["routing"], 16, 2, 2)
    assert np.allclose(res["O"][0], ref, atol=1e-12)
    sizes = [res["routing"][(0, 0, i)].support.size for i in range(n)]
    assert min(sizes) == 0 and max(sizes) >= 2           # chunk-0 rows route nothing; later rows do
    assert any(0 < s < i // 16 for i, s in enumerate(sizes))   # and the threshold really prunes


def test_everything_selected_and_weak_prior_is_dense_causal_attention():
    """gamma -> 0 makes entmax uniform (every visible chunk routed); with sigma large the bias
    vanishes, so the output is plain causal softmax attention."""
    Q, K, V = _case(40, n=96, scale=1.0)
    res = orc.forward_prefill(Q, K, V, B=16, alpha=1.5, gamma=1e-6, sigma=1e9)
    for i in range(96):
        assert res["routing"][(0, 0, i)].support.size == i // 16
    for h in range(4):
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q[0, :, h])[None], torch.from_numpy(K[0, :, h // 2])[None],
            torch.from_numpy(V[0, :, h // 2])[None], is_causal=True)[0].numpy()
        assert np.allclose(res["O"][0, :, h], ref, atol=1e-9)


def test_large_sigma_is_plain_softmax_over_selected_tokens():
    Q, K, V = _case(50)
    Kbar = orc.block_summaries(K[0], 16)
    rt, o = orc.forward_row(Q[0], K[0], V[0], Kbar, 150, 1, B=16, alpha=1.5, gamma=3.0, sigma=1e12)
    o0 = orc.attend_row(Q[0, 150, 2:4], K[0, :, 1], V[0, :, 1], 16, rt.support, np.zeros(rt.support.size), 144, 151)
    assert np.allclose(o, o0, atol=1e-10)


def test_decode_equals_last_prefill_row_and_ignores_cache_tail():
    Q, K, V = _case(60, n=150)
    pre = orc.forward_prefill(Q, K, V, B=16, alpha=1.5, gamma=3.0, sigma=5.0, rows=[99, 149])
    for L in (100, 150):
        dec = orc.forward_decode(Q[:, L - 1], K, V, [L], B=16, alpha=1.5, gamma=3.0, sigma=5.0)
        assert np.allclose(dec["O"][0], pre["O"][0, L - 1], atol=1e-13)
        assert np.array_equal(dec["routing"][(0, 1)].support, pre["routing"][(0, 1, L - 1)].support)


def test_non_causal_reading_against_dense_masked_attention():
    Q, K, V = _case(70, n=70)
    B = 16
    res = orc.forward_prefill(Q, K, V, B=B, alpha=1.5, gamma=3.0, sigma=2.0, causal=False)
    for r in range(2):
        for i in (0, 33, 69):
            rt = res["routing"][(0, r, i)]
            assert rt.n_cand == 4
            M = np.full(70, -np.inf)
            for c, dc in zip(rt.support, rt.bias):
                M[c * B:(c + 1) * B] = dc
            M[64:70] = 0.0
            for h in (2 * r, 2 * r + 1):
                z = K[0, :, r] @ Q[0, i, h] / math.sqrt(8) + M
                p = np.exp(z - z.max())
                p /= p.sum()
                assert np.allclose(res["O"][0, i, h], p @ V[0, :, r], atol=1e-12)


def test_mask_packing_and_statistics():
    w = orc.pack_mask_words(np.array([0, 31, 32, 70]), 95, 3)
    assert list(w) == [0x80000001, 0x00000001, (1 << 6) | (1 << 31)]
    assert orc.block_sparsity([0, 1, 2], [0, 3, 8]) == pytest.approx(1 - 6 / 14)
    assert orc.selected_flops([2], [5], 64, 128, 4) == 4 * 128 * 4 * (128 + 5)


# ------------------------------------------------------------------ local window (diagonal + previous chunks)

def test_local_window_zero_is_the_printed_algorithms():
    Q, K, V = _case(80, n=120)
    a = orc.forward_prefill(Q, K, V, B=16, alpha=1.5, gamma=3.0, sigma=2.0)
    b = orc.forward_prefill(Q, K, V, B=16, alpha=1.5, gamma=3.0, sigma=2.0, local_blocks=0)
    assert np.array_equal(a["O"], b["O"])
    assert all(rt.local.size == 0 for rt in b["routing"].values())


@pytest.mark.parametrize("L", [1, 2, 3])
def test_local_window_against_dense_masked_attention(L):
    """Token-level brute force: the window chunks and the causal part of the diagonal chunk get bias 0, the
    routed chunks (all before the window) their bias, everything else -inf; softmax written out here."""
    Q, K, V = _case(81, n=150)
    B, d = 16, 8
    res = orc.forward_prefill(Q, K, V, B=B, alpha=1.5, gamma=3.0, sigma=2.0, local_blocks=L)
    routed_any = False
    for r in range(2):
        for i in range(150):
            rt = res["routing"][(0, r, i)]
            c_i = i // B
            lo = max(c_i - L, 0)
            assert rt.n_cand == lo and list(rt.local) == list(range(lo, c_i))
            assert all(c < lo for c in rt.support)
            routed_any |= rt.support.size > 0
            M = np.full(150, -np.inf)
            for c, dc in zip(rt.support, rt.bias):
                M[c * B:(c + 1) * B] = dc
            M[lo * B:i + 1] = 0.0
            for h in (2 * r, 2 * r + 1):
                z = K[0, :, r] @ Q[0, i, h] / math.sqrt(d) + M
                p = np.exp(z - z.max())
                p /= p.sum()
                assert np.allclose(res["O"][0, i, h], p @ V[0, :, r], atol=1e-12)
    assert routed_any


def test_local_window_covering_everything_is_dense_causal_attention():
    """A window at least as long as the sequence leaves nothing to route: the result is plain causal softmax
    attention whatever alpha, gamma and sigma are."""
    Q, K, V = _case(82, n=96, scale=1.0)
    res = orc.forward_prefill(Q, K, V, B=16, alpha=1.25, gamma=5.0, sigma=0.5, local_blocks=6)
    for h in range(4):
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Q[0, :, h])[None], torch.from_numpy(K[0, :, h // 2])[None],
            torch.from_numpy(V[0, :, h // 2])[None], is_causal=True)[0].numpy()
        assert np.allclose(res["O"][0, :, h], ref, atol=1e-12)
    assert all(rt.n_cand == 0 for rt in res["routing"].values())


@pytest.mark.parametrize("sigma", [1.0, 10.0, 1e8])
def test_local_window_bias_form_equals_definition_form(sigma):
    """Proposition 1 with |D_i| = window tokens + causal diagonal tokens (Eq. 9-10 count tokens)."""
    Q, K, V = _case(83)
    B = 16
    Kbar = orc.block_summaries(K[0], B)
    for L in (1, 2):
        for i in (15, 16, 40, 63, 100, 199):
            for r in (0, 1):
                rt, o = orc.forward_row(Q[0], K[0], V[0], Kbar, i, r, B=B, alpha=1.5, gamma=3.0, sigma=sigma,
                                        local_blocks=L)
                lo = max(i // B - L, 0)
                o2 = orc.attend_row_definition_form(Q[0, i, 2 * r:2 * r + 2], K[0, :, r], V[0, :, r], B,
                                                    rt.support, rt.w[rt.support] if rt.n_cand else np.zeros(0),
                                                    sigma, lo * B, i + 1)
                assert np.allclose(o, o2, rtol=1e-11, atol=1e-12)


def test_local_window_size_matches_the_training_setting():
    """B = 64, one window chunk: D_i holds 64 + (i mod 64) + 1 tokens once a previous chunk exists (the
    appendix's "64-127 tokens" counts the positions before the query)."""
    for i in (64, 100, 127, 128, 1000):
        n_cand, dlo, dhi = orc._row_geometry(i, 4096, 64, True, 1)
        assert dhi - dlo - 1 == 64 + i % 64 and 64 <= dhi - dlo - 1 <= 127
        assert n_cand == i // 64 - 1


def test_local_window_decode_equals_last_prefill_row():
    Q, K, V = _case(84, n=150)
    pre = orc.forward_prefill(Q, K, V, B=16, alpha=1.5, gamma=3.0, sigma=5.0, rows=[99, 149], local_blocks=2)
    for L in (100, 150):
        dec = orc.forward_decode(Q[:, L - 1], K, V, [L], B=16, alpha=1.5, gamma=3.0, sigma=5.0, local_blocks=2)
        assert np.allclose(dec["O"][0], pre["O"][0, L - 1], atol=1e-13)
        assert np.array_equal(dec["routing"][(0, 1)].local, pre["routing"][(0, 1, L - 1)].local)


def test_local_window_is_causal_only():
    Q, K, V = _case(85, n=64)
    with pytest.raises(ValueError):
        orc.forward_prefill(Q, K, V, B=16, alpha=1.5, causal=False, local_blocks=1)
