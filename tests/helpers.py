"""Test helpers: run the oracle on seeded inputs and compare the CUDA library's outputs with it."""
from __future__ import annotations

import numpy as np
import torch

from oracle import dash_oracle as orc

BORDERLINE = 1e-4      # |margin| below which a chunk's membership may legitimately differ (score units)


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def tol_for(dtype: torch.dtype):
    """(max-abs, mean-abs) output tolerance: bf16 2e-2 / 2e-3, fp32 1e-4 / 1e-5."""
    return (2e-2, 2e-3) if dtype == torch.bfloat16 else (1e-4, 1e-5)


def oracle_prefill_rows(Q, K, V, *, B, alpha, gamma, sigma, rows, kv_heads=None, batches=None, qbar=None,
                        local_blocks=0, causal=True):
    """Oracle routing + outputs for the given rows.  Returns dict[(b, r, i)] -> (RowRouting, O [g_q, d])."""
    Qn, Kn, Vn = to_np64(Q), to_np64(K), to_np64(V)
    b, n, h_q, d = Qn.shape
    h_kv = Kn.shape[2]
    out = {}
    for bb in (range(b) if batches is None else batches):
        Kbar = orc.block_summaries(Kn[bb], B, qbar)
        for r in (range(h_kv) if kv_heads is None else kv_heads):
            for i in rows:
                out[(bb, r, int(i))] = orc.forward_row(Qn[bb], Kn[bb], Vn[bb], Kbar, int(i), r, B=B, alpha=alpha,
                                                       gamma=gamma, sigma=sigma, local_blocks=local_blocks,
                                                       causal=causal)
    return out


def routing_to_abi(routing: dict, p, list_offset_fn, device="cuda"):
    """Packs oracle routing of ALL rows into the mask / count / list layout of the C ABI."""
    T_a = (p.seq_kv + p.block - 1) // p.block
    W = (T_a + 31) // 32
    mask = np.zeros((p.batch, p.h_kv, p.seq_q, W), dtype=np.uint32)
    count = np.zeros((p.batch, p.h_kv, p.seq_q), dtype=np.int32)
    cap = max(int(list_offset_fn(p, p.batch - 1, p.h_kv - 1, p.seq_q - 1)) + T_a, 1)
    idx = np.zeros(cap, dtype=np.int32)
    bias = np.zeros(cap, dtype=np.float32)
    for (b, r, i), val in routing.items():
        rt = val[0] if isinstance(val, tuple) else val
        own = i // p.block if p.seq_q > 1 else None
        # window chunks close the list as ordinary entries with bias 0 (their bits set, counted), as the ABI states
        members = np.concatenate([rt.support, rt.local]).astype(np.int64)
        mask[b, r, i if p.seq_q > 1 else 0] = orc.pack_mask_words(members, own, W)
        count[b, r, i if p.seq_q > 1 else 0] = members.size
        off = int(list_offset_fn(p, b, r, i if p.seq_q > 1 else 0))
        idx[off:off + members.size] = members
        bias[off:off + rt.support.size] = rt.bias
        bias[off + rt.support.size:off + members.size] = 0.0
    dev = lambda a: torch.from_numpy(a.view(np.int32) if a.dtype == np.uint32 else a).to(device)
    return dev(mask), dev(count), dev(idx), dev(bias)


def compare_routing(rt: orc.RowRouting, own_chunk, mask_words: np.ndarray, count: int, bias_list: np.ndarray,
                    idx_list, sigma: float, exponent: float):
    """Checks one row's GPU routing against the oracle.  Returns (n_borderline, n_differing, clean) where
    `clean` says the supports are identical (so outputs are comparable); exponent = 1/(alpha-1)."""
    W = mask_words.size
    got = set()
    for w in range(W):
        word = int(mask_words[w]) & 0xFFFFFFFF
        while word:
            bit = (word & -word).bit_length() - 1
            got.add(w * 32 + bit)
            word &= word - 1
    if own_chunk is not None:
        assert own_chunk in got, "own chunk's bit must be set"
        got.discard(own_chunk)
    # window chunks (local_blocks > 0): bits set, listed behind the routed chunks with bias exactly 0, counted
    local = [int(c) for c in rt.local]
    assert set(local) <= got, "every window chunk's bit must be set"
    got -= set(local)
    assert count >= len(local), "count includes the window chunks"
    count -= len(local)
    if local:
        assert (np.asarray(bias_list[count:count + len(local)]) == 0.0).all(), "window chunks carry bias 0"
        if idx_list is not None:
            assert list(idx_list[count:count + len(local)]) == local, "window chunks close the list in order"
    want = set(int(c) for c in rt.support)
    border = set(int(c) for c in np.nonzero(np.abs(rt.margin) <= BORDERLINE)[0]) if rt.n_cand else set()
    diff = got ^ want
    assert diff <= border, f"support differs outside the borderline band: {sorted(diff - border)[:8]}"
    assert count == len(got), "count must equal the number of routed bits"
    if idx_list is not None:
        assert list(idx_list[:count]) == sorted(got), "block list must be the ascending routed chunks"
    clean = not diff
    if clean and count:
        # log w = e*log(margin) + ...: an fp32 margin error delta moves log w by about e*delta/margin, and
        # the mean mu by the mean of those; compare only rows without a borderline member
        if not (border & want):
            delta = 3e-5 * max(1.0, float(np.abs(rt.x).max()))
            per = exponent * delta / rt.margin[rt.support]
            tol = (per + per.mean()) / sigma + 2e-6
            err = np.abs(bias_list[:count] - rt.bias)
            assert (err <= tol).all(), f"bias error {err.max()} (tolerance {tol[np.argmax(err - tol)]})"
    return len(border), len(diff), clean


def check_outputs(got: np.ndarray, want: np.ndarray, dtype: torch.dtype, what=""):
    mx, mean = tol_for(dtype)
    err = np.abs(got - want)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    assert err.max() <= mx, f"{what}: max-abs {err.max():.3e} > {mx}"
    assert err.mean() <= mean, f"{what}: mean-abs {err.mean():.3e} > {mean}"
    return float(err.max()), float(err.mean())
