"""Device-side error reporting without a GPU fault: the status word is sticky, and while it holds an error the
tensor-core kernels retire at their first wait instead of computing.  The error is made on the host (the word
is written from the host); nothing on the GPU is made to hang, trap or fault."""
import time

import pytest
import torch

from paper_2605_18753_b200 import binding as B
from paper_2605_18753_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"
DASH_ERR_TIMEOUT = -7


def _set_status(ws, code):
    ws[:4].copy_(torch.tensor([code], dtype=torch.int32).view(torch.uint8))
    torch.cuda.synchronize()


def test_status_word_is_sticky_and_reset_restores_service():
    w = synth.workload("prefill_8k", seq=2048)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    O = torch.empty_like(Q)
    p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    ws = B.alloc_workspace(p)
    B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
    assert B.dash_attn_last_status(ws) == 0
    good = O.clone()

    _set_status(ws, DASH_ERR_TIMEOUT)            # as if a bounded wait had run out in an earlier kernel
    O.fill_(float("nan"))
    t0 = time.time()
    B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
    assert B.dash_attn_last_status(ws) == DASH_ERR_TIMEOUT      # first error wins, nothing overwrites it
    assert time.time() - t0 < 5.0                # no block sat out a wait limit

    B.dash_attn_reset_status(ws)
    B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
    assert B.dash_attn_last_status(ws) == 0
    assert torch.equal(O, good)                  # the path is deterministic


def test_status_word_decode_path():
    w = synth.workload("decode_128k", batch=2, seq=8192)
    di = synth.make_decode_inputs(w, DEV)
    q, Kc, Vc, kl = di["Q"], di["K"], di["V"], di["kv_len"]
    o = torch.empty_like(q)
    p = B.params_for_decode(q, Kc, Vc, o, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    kbar = B.alloc_kbar(p)
    B.dash_attn_block_summaries(p, Kc, kbar, kv_len=kl)
    ws = B.alloc_workspace(p)
    B.dash_attn_fwd_decode(p, q, Kc, Vc, kbar, kl, o, ws)
    assert B.dash_attn_last_status(ws) == 0
    good = o.clone()
    _set_status(ws, DASH_ERR_TIMEOUT)
    B.dash_attn_fwd_decode(p, q, Kc, Vc, kbar, kl, o, ws)
    assert B.dash_attn_last_status(ws) == DASH_ERR_TIMEOUT
    B.dash_attn_reset_status(ws)
    B.dash_attn_fwd_decode(p, q, Kc, Vc, kbar, kl, o, ws)
    assert B.dash_attn_last_status(ws) == 0
    assert torch.equal(o, good)


def test_bounded_wait_really_runs_out_and_the_kernel_returns():
    """A device-side wait that nothing will ever satisfy: through the test hooks the prefill attention kernel is told
    not to issue the load of its first K tile and to give up a wait after 2e5 cycles (0.1 ms).  The waits for that tile
    run out, every role leaves its loop, the copies in flight land, tensor memory is freed and the kernel returns
    with DASH_ERR_TIMEOUT in the status word -- no hang, no trap, no fault -- and after a reset the same workspace
    serves a correct forward pass again."""
    w = synth.workload("prefill_8k", seq=1024)
    inp = synth.make_prefill_inputs(w, DEV)
    Q, K, V = inp["Q"], inp["K"], inp["V"]
    O = torch.empty_like(Q)
    p = B.params_for_prefill(Q, K, V, O, block=w.block, alpha=w.alpha, gamma=w.gamma, sigma=w.sigma)
    ws = B.alloc_workspace(p)
    B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
    assert B.dash_attn_last_status(ws) == 0
    good = O.clone()
    try:
        B.dash_attn_test_hooks(wait_limit_cycles=200_000, skip_own_k_load=1)
        O.fill_(float("nan"))
        t0 = time.time()
        B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
        assert B.dash_attn_last_status(ws) == DASH_ERR_TIMEOUT
        assert time.time() - t0 < 5.0            # one short wait limit, then the rest of the grid retires at once
    finally:
        B.dash_attn_test_hooks()                 # defaults
    torch.cuda.synchronize()                     # the context is intact: nothing faulted
    B.dash_attn_reset_status(ws)
    B.dash_attn_fwd_prefill(p, Q, K, V, O, ws)
    assert B.dash_attn_last_status(ws) == 0
    assert torch.equal(O, good)
