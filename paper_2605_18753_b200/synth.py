"""Seeded synthetic workloads (inputs only; none of the method's arithmetic lives here).

Two recipes:

* ``tiny``: Q, K, V i.i.d. N(0,1)/sqrt(d) in fp32.
* ``planted``: per (batch, KV head) a unit direction u; queries are
  rho*sqrt(d)*u + N(0, I); keys and values are N(0, I); ``n_planted`` complete
  chunks per (batch, KV head), drawn without replacement, have their keys moved
  by ``shift * u`` ("toward the query mean").  A planted chunk's summary scores
  about rho*shift against every query of the group, an ordinary chunk scores
  N(0, (rho^2+1)/B); rho and shift set how many ordinary chunks survive the
  entmax threshold, i.e. the block sparsity.

Every tensor draws from its own ``torch.Generator`` seeded ``seed*1000 + k`` so
that a tensor's values do not depend on the shapes of the others.  Generation
runs on the requested device (CPU for tests against the oracle at small sizes,
the GPU for full-size workloads, which are then copied to the host for the
oracle's sampled rows).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, asdict, replace

import torch

__all__ = ["Workload", "WORKLOADS", "make_prefill_inputs", "make_decode_inputs", "workload"]


@dataclass(frozen=True)
class Workload:
    name: str
    kind: str            # "prefill" | "decode"
    batch: int
    seq: int             # prefill: n; decode: KV length including the new token
    h_q: int
    h_kv: int
    head_dim: int
    block: int
    alpha: float
    dtype: str           # "f32" | "bf16"
    recipe: str          # "tiny" | "planted"
    gamma: float = 1.0
    sigma: float = 10.0
    rho: float = 0.72
    shift: float = 2.0
    n_planted: int = 8
    seed: int = 0
    q_corr: float = 0.0  # AR(1) coefficient of the query noise along the token axis (0 = independent queries)

    def as_dict(self):
        return asdict(self)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


# rho / shift values are the frozen results of the calibration script that
# sits beside the oracle (achieved sparsities are recorded in
# tests/golden/calibration.json).
WORKLOADS = {
    # C1: tiny fp32 check; gamma=1 selects every visible chunk (scores ~1e-3 apart)
    "tiny": Workload("tiny", "prefill", 1, 1024, 1, 1, 64, 64, 1.5, "f32", "tiny"),
    # C1': same tensors, gamma large enough that the threshold actually prunes
    "tiny_g512": Workload("tiny_g512", "prefill", 1, 1024, 1, 1, 64, 64, 1.5, "f32", "tiny", gamma=512.0),
    # C2: prefill 8K, ~75 % block sparsity
    "prefill_8k": Workload("prefill_8k", "prefill", 1, 8192, 32, 8, 128, 64, 1.5, "bf16", "planted",
                           rho=0.72, shift=2.0),
    # the 8K prefill with the finer chunks of the paper's chunk-size study (its sparsities there: 75.7 % at 32,
    # 77.0 % at 16); same tensors' recipe, shift re-calibrated for chunks of 16
    "prefill_8k_b32": Workload("prefill_8k_b32", "prefill", 1, 8192, 32, 8, 128, 32, 1.5, "bf16", "planted",
                               rho=0.72, shift=1.78),
    "prefill_8k_b16": Workload("prefill_8k_b16", "prefill", 1, 8192, 32, 8, 128, 16, 1.5, "bf16", "planted",
                               rho=0.72, shift=1.77),
    # C3: prefill 64K at ~75 % and ~90 %
    "prefill_64k_s75": Workload("prefill_64k_s75", "prefill", 1, 65536, 32, 8, 128, 64, 1.5, "bf16", "planted",
                                rho=0.72, shift=1.56),
    "prefill_64k_s90": Workload("prefill_64k_s90", "prefill", 1, 65536, 32, 8, 128, 64, 1.5, "bf16", "planted",
                                rho=0.72, shift=2.10),
    # C4: decode, batch 16, 131072-token cache, ~90 %
    "decode_128k": Workload("decode_128k", "decode", 16, 131072, 32, 8, 128, 64, 1.5, "bf16", "planted",
                            rho=0.72, shift=1.42),
    # C5: alpha sweep base point (block and alpha are varied by the caller)
    "sweep_32k": Workload("sweep_32k", "prefill", 2, 32768, 32, 8, 128, 64, 1.5, "bf16", "planted",
                          rho=0.72, shift=2.0),
}


def workload(name: str, **overrides) -> Workload:
    w = WORKLOADS[name]
    return w.with_(**overrides) if overrides else w


def _gen(seed: int, k: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed * 1000 + k)
    return g


def _torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _planted_parts(w: Workload, n_tokens: int, device):
    """Directions [b, h_kv, d] and planted chunk ids [b, h_kv, n_planted]."""
    b, h_kv, d = w.batch, w.h_kv, w.head_dim
    u = torch.randn(b, h_kv, d, generator=_gen(w.seed, 0, device), device=device, dtype=torch.float32)
    u = u / u.norm(dim=-1, keepdim=True)
    T_s = n_tokens // w.block
    n_pl = min(w.n_planted, T_s)
    gp = _gen(w.seed, 1, "cpu")
    planted = torch.stack([torch.stack([torch.randperm(T_s, generator=gp)[:n_pl] for _ in range(h_kv)])
                           for _ in range(b)]) if n_pl > 0 else torch.zeros(b, h_kv, 0, dtype=torch.long)
    return u, planted.to(device)


def _keys_values(w: Workload, n_tokens: int, u, planted, device):
    b, h_kv, d, B = w.batch, w.h_kv, w.head_dim, w.block
    dt = _torch_dtype(w.dtype)
    K = torch.empty(b, n_tokens, h_kv, d, device=device, dtype=dt)
    V = torch.empty(b, n_tokens, h_kv, d, device=device, dtype=dt)
    gk, gv = _gen(w.seed, 2, device), _gen(w.seed, 3, device)
    for bb in range(b):                      # one sequence at a time bounds the fp32 temporaries
        k32 = torch.randn(n_tokens, h_kv, d, generator=gk, device=device, dtype=torch.float32)
        for r in range(h_kv):
            for c in planted[bb, r].tolist():
                k32[c * B:(c + 1) * B, r, :] += w.shift * u[bb, r]
        K[bb] = k32.to(dt)
        del k32
        V[bb] = torch.randn(n_tokens, h_kv, d, generator=gv, device=device, dtype=torch.float32).to(dt)
    return K, V


def _ar1_along_tokens(x: torch.Tensor, c: float) -> torch.Tensor:
    """x[i] <- c x[i-1] + sqrt(1 - c^2) x[i] along dim 0 (x[0] kept): unit variance, lag-1 correlation c.

    Evaluated segment by segment as a scaled cumulative sum in float64 (c^-L stays below 1e6 inside a segment)."""
    if c <= 0.0:
        return x
    n = x.shape[0]
    L = max(1, min(n, int(13.8 / -math.log(c))))
    s = math.sqrt(1.0 - c * c)
    out = torch.empty_like(x)
    prev = None
    for a in range(0, n, L):
        seg = x[a:a + L].to(torch.float64) * s
        if prev is None:
            seg[0] = x[0].to(torch.float64)
        t = torch.arange(seg.shape[0], device=x.device, dtype=torch.float64)
        up = (c ** t).view(-1, *([1] * (x.dim() - 1)))
        acc = torch.cumsum(seg / up, dim=0) * up
        if prev is not None:
            acc = acc + up * c * prev
        prev = acc[-1]
        out[a:a + L] = acc.to(x.dtype)
    return out


def make_prefill_inputs(w: Workload, device="cpu"):
    """Returns dict(Q [b,n,h_q,d], K [b,n,h_kv,d], V, planted [b,h_kv,n_planted])."""
    assert w.kind == "prefill"
    b, n, h_q, h_kv, d = w.batch, w.seq, w.h_q, w.h_kv, w.head_dim
    dt = _torch_dtype(w.dtype)
    if w.recipe == "tiny":
        s = 1.0 / math.sqrt(d)
        mk = lambda k, h: (torch.randn(b, n, h, d, generator=_gen(w.seed, k, device), device=device,
                                       dtype=torch.float32) * s).to(dt)
        return {"Q": mk(0, h_q), "K": mk(1, h_kv), "V": mk(2, h_kv),
                "planted": torch.zeros(b, h_kv, 0, dtype=torch.long)}
    u, planted = _planted_parts(w, n, device)
    K, V = _keys_values(w, n, u, planted, device)
    g_q = h_q // h_kv
    Q = torch.empty(b, n, h_q, d, device=device, dtype=dt)
    gq = _gen(w.seed, 4, device)
    for bb in range(b):
        q32 = torch.randn(n, h_q, d, generator=gq, device=device, dtype=torch.float32)
        q32 = _ar1_along_tokens(q32, w.q_corr)
        q32 += (w.rho * math.sqrt(d)) * u[bb].repeat_interleave(g_q, dim=0)[None, :, :]
        Q[bb] = q32.to(dt)
        del q32
    return {"Q": Q, "K": K, "V": V, "planted": planted}


def make_decode_inputs(w: Workload, device="cpu", kv_len=None):
    """Returns dict(Q [b,h_q,d], K/V cache [b,cap,h_kv,d], kv_len int32 [b], planted).

    ``kv_len`` (list of ints) defaults to the full capacity ``w.seq`` for every
    sequence; shorter entries leave the cache tail filled but unused.
    """
    assert w.kind == "decode"
    b, cap, h_q, h_kv, d = w.batch, w.seq, w.h_q, w.h_kv, w.head_dim
    dt = _torch_dtype(w.dtype)
    u, planted = _planted_parts(w, cap, device)
    K, V = _keys_values(w, cap, u, planted, device)
    g_q = h_q // h_kv
    q32 = torch.randn(b, h_q, d, generator=_gen(w.seed, 4, device), device=device, dtype=torch.float32)
    q32 += (w.rho * math.sqrt(d)) * u.repeat_interleave(g_q, dim=1)
    lens = torch.full((b,), cap, dtype=torch.int32) if kv_len is None else torch.tensor(kv_len, dtype=torch.int32)
    assert lens.numel() == b and int(lens.max()) <= cap and int(lens.min()) >= 1
    return {"Q": q32.to(dt), "K": K, "V": V, "kv_len": lens.to(device), "planted": planted}
