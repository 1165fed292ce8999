"""The seeded input generators (no method arithmetic lives there): determinism and the correlated-query option."""
import math

import torch

from paper_2605_18753_b200 import synth


def test_generators_are_deterministic_and_seeded():
    w = synth.workload("prefill_8k", seq=512)
    a, b = synth.make_prefill_inputs(w), synth.make_prefill_inputs(w)
    for k in ("Q", "K", "V"):
        assert torch.equal(a[k], b[k])
    c = synth.make_prefill_inputs(w.with_(seed=1))
    assert not torch.equal(a["Q"], c["Q"])


def test_query_correlation_is_an_ar1_filter_and_off_by_default():
    x = torch.randn(3000, 2, 4, generator=torch.Generator().manual_seed(0))
    assert synth._ar1_along_tokens(x, 0.0) is x
    for c in (0.5, 0.99):
        y = synth._ar1_along_tokens(x, c)
        z = x.clone().double()
        s = math.sqrt(1 - c * c)
        for i in range(1, x.shape[0]):
            z[i] = c * z[i - 1] + s * x[i].double()
        assert float((y.double() - z).abs().max()) < 1e-5
        assert 0.8 < float(y.var()) < 1.2
    w = synth.workload("prefill_8k", seq=512)
    assert w.q_corr == 0.0
    q0 = synth.make_prefill_inputs(w)["Q"]
    q1 = synth.make_prefill_inputs(w.with_(q_corr=0.99))["Q"]
    assert not torch.equal(q0, q1)
    # neighbouring queries agree far more than independent ones
    def lag1(q):
        q = q[0].float()
        q = q - q.mean(dim=0, keepdim=True)       # remove the planted direction common to all tokens
        return float((q[1:] * q[:-1]).sum() / (q * q).sum())
    assert lag1(q1) > 0.9 and abs(lag1(q0)) < 0.1
