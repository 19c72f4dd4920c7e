"""The autograd front end and the end-to-end layer case (config 5).  GPU only."""
import numpy as np
import pytest

from paper_2512_13368_b200 import workloads
from parity_util import tolerance

pytestmark = pytest.mark.gpu


def test_autograd_matches_oracle():
    import torch
    import oracle
    from paper_2512_13368_b200.autograd import blossom_attention
    w = workloads.make("autograd", "bf16", 2, 2, 320, 32, 32, 3, 48, seed=21)
    dev = torch.device("cuda:0")
    t = lambda a: torch.from_numpy(a).to(dev).to(torch.bfloat16).requires_grad_(True)  # noqa: E731
    q, k, v = t(w.q), t(w.k), t(w.v)
    gate = torch.from_numpy(w.gate).to(dev).requires_grad_(True)
    out, idx = blossom_attention(q, k, v, gate, w.block, w.topk, w.window, return_indices=True)
    out.backward(torch.from_numpy(w.dout).to(dev).to(torch.bfloat16))
    ref = oracle.forward_backward(w.q, w.k, w.v, w.gate, w.dout, w.block, w.topk, w.window, None,
                                  idx=idx.cpu().numpy())
    got = {"out": out, "dq": q.grad, "dk": k.grad, "dv": v.grad, "dgate": gate.grad}
    for key, val in got.items():
        err = float(np.abs(val.detach().float().cpu().numpy() - ref[key]).max())
        assert err <= tolerance(w, ref[key]), (key, err)


def test_layer_step_runs_and_reports_attention_share():
    from paper_2512_13368_b200 import layer_step
    r = layer_step.attention_share(batch=8, seq_len=256, n_items=2000, negatives=15, steps=2, warmup=1)
    assert np.isfinite(r["loss"]) and r["loss"] > 0
    assert 0.0 < r["attention_share"] < 1.0
    assert r["library_launches_per_step"] >= 2 * 7   # two layers x (selection, forward, backward kernels)
