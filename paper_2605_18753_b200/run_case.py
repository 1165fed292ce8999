"""Runs one synthetic workload through the library a few times and prints CUDA-event timings.

    python -m paper_2605_18753_b200.run_case prefill_8k --iters 5
    python -m paper_2605_18753_b200.run_case decode_128k --batch 4 --iters 3      # 2 GiB of KV cache instead of 8
    python -m paper_2605_18753_b200.run_case prefill_8k --backward --iters 2       # Stage-2 backward on tensor cores

A quick way to see the path work on a given shape (overrides: --batch, --seq, --block, --alpha, --head-dim, --local-blocks), and a small,
self-terminating command to put under a profiler.  Inputs are the seeded synthetic tensors of `synth`."""
from __future__ import annotations

import argparse

import torch

from . import binding as B
from . import synth


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("workload", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--iters", type=int, default=5)
    ap.add_argument("--batch", type=int)
    ap.add_argument("--seq", type=int)
    ap.add_argument("--block", type=int)
    ap.add_argument("--alpha", type=float)
    ap.add_argument("--head-dim", type=int, dest="head_dim")
    ap.add_argument("--local-blocks", type=int, default=0, help="window chunks before the own chunk (0 = none)")
    ap.add_argument("--backward", action="store_true", help="prefill only: time the tensor-core Stage-2 backward instead")
    args = ap.parse_args()
    over = {k: getattr(args, k) for k in ("batch", "seq", "block", "alpha", "head_dim") if getattr(args, k) is not None}
    w = synth.workload(args.workload, **over)
    dev = "cuda"
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)     # larger than L2

    if w.kind == "prefill":
        inp = synth.make_prefill_inputs(w, dev)
        Q, K, V = inp["Q"], inp["K"], inp["V"]
        O = torch.empty_like(Q)
        p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma,
                                 local_blocks=args.local_blocks)
        ws = B.alloc_workspace(p)
        step = lambda: B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
        if args.backward:
            # routing from one forward pass, then the gradients of Stage 2 for a random dO
            rt, kbar = B.alloc_routing(p), B.alloc_kbar(p)
            B.dash_attn_block_summaries(p, K, kbar)
            B.dash_attn_select(p, Q, kbar, rt["mask"], rt["count"], rt["blk_idx"], rt["blk_bias"], ws)
            dO = torch.randn(Q.shape, device=dev, dtype=torch.float32).to(Q.dtype)
            dQ = torch.empty_like(Q)
            dK = torch.empty(w.batch, w.seq, w.h_kv, w.head_dim, device=dev)
            dV = torch.empty_like(dK)
            dbias = torch.empty_like(rt["blk_bias"])
            ws = B.alloc_bwd_workspace(p)        # its status word is the one checked below
            O = dQ
            step = lambda: B.dash_attn_bwd_attend_prefill_tc(p, Q, K, V, dO, rt["mask"], rt["blk_bias"], dQ, dK, dV, dbias, ws)
    else:
        di = synth.make_decode_inputs(w, dev)
        q, Kc, Vc, kl = di["Q"], di["K"], di["V"], di["kv_len"]
        del di
        O = torch.empty_like(q)
        p = B.params_for_decode(q, Kc, Vc, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma,
                                local_blocks=args.local_blocks)
        kbar = B.alloc_kbar(p)
        B.dash_attn_block_summaries(p, Kc, kbar, kv_len=kl)
        ws = B.alloc_workspace(p)
        step = lambda: B.dash_attn_fwd_decode(p, q, Kc, Vc, kbar, kl, O, ws)

    times = []
    for it in range(args.iters + 1):
        flush.fill_(it & 1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        step()
        b.record()
        torch.cuda.synchronize()
        if it > 0:
            times.append(a.elapsed_time(b))
    status = B.dash_attn_last_status(ws)
    print(f"{w.name} {over or ''}: {'backward' if args.backward else 'forward'} ms {['%.4f' % t for t in times]}  status {B.STATUS.get(status, status)}  "
          f"output finite {bool(torch.isfinite(O.float()).all())}")
    if status != 0:
        raise SystemExit(1)


if __name__ == "__main__":
    main()
