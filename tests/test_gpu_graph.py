"""The entry points enqueue kernels on the caller's stream and allocate nothing, so a forward pass can be
recorded into a CUDA graph and replayed: the replay must reproduce the eager result bit for bit, also after the
inputs changed in place (the graph holds pointers, not values)."""
import pytest
import torch

from paper_2605_18753_b200 import binding as B
from paper_2605_18753_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _capture(step):
    step()                                   # first use outside the capture (per-kernel attributes, tensor-map encoder)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    return g


def test_prefill_forward_replays_from_a_cuda_graph():
    w = synth.workload("prefill_8k", seq=3000)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    O = torch.empty_like(Q)
    p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma, local_blocks=1)
    ws = B.alloc_workspace(p)
    g = _capture(lambda: B.dash_attn_fwd_prefill(p, Q, K, V, O, ws))
    eager = O.clone()
    O.fill_(float("nan"))
    g.replay()
    torch.cuda.synchronize()
    assert B.dash_attn_last_status(ws) == 0
    assert torch.equal(O, eager)
    # new inputs in the same buffers
    inp2 = synth.make_prefill_inputs(w.with_(seed=5), DEV)
    Q.copy_(inp2["Q"]); K.copy_(inp2["K"]); V.copy_(inp2["V"])
    g.replay()
    torch.cuda.synchronize()
    replayed = O.clone()
    B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
    torch.cuda.synchronize()
    assert torch.equal(O, replayed) and not torch.equal(O, eager)


def test_decode_step_replays_from_a_cuda_graph():
    w = synth.workload("decode_128k", batch=2, seq=20000)
    di = synth.make_decode_inputs(w, DEV, kv_len=[20000, 12345])
    q, Kc, Vc, kl = di["Q"], di["K"], di["V"], di["kv_len"]
    O = torch.empty_like(q)
    p = B.params_for_decode(q, Kc, Vc, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, Kc, kbar, kv_len=kl)
    ws = B.alloc_workspace(p)
    g = _capture(lambda: B.dash_attn_fwd_decode(p, q, Kc, Vc, kbar, kl, O, ws))
    eager = O.clone()
    for _ in range(3):                       # the arrival counters clear themselves: replays can follow each other
        O.fill_(float("nan"))
        g.replay()
    torch.cuda.synchronize()
    assert B.dash_attn_last_status(ws) == 0
    assert torch.equal(O, eager)
    kl.copy_(torch.tensor([15000, 777], dtype=kl.dtype))      # the lengths live on the device: a replay sees them
    g.replay()
    torch.cuda.synchronize()
    replayed = O.clone()
    B.dash_attn_fwd_decode(p, q, Kc, Vc, kbar, kl, O, ws)
    torch.cuda.synchronize()
    assert torch.equal(O, replayed) and not torch.equal(O, eager)
