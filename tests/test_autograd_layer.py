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


def test_autograd_packed_projection_views_and_grouped_heads():
    """q, k, v cut out of one packed projection buffer (equal strides, not dense: the layout that
    once made the outputs overrun their allocation), int64 lengths, and 4 query heads on 2
    key/value heads: outputs and gradients against the oracle."""
    import torch
    import oracle
    from paper_2512_13368_b200.autograd import blossom_attention
    dev = torch.device("cuda:0")
    bf = lambda a: torch.from_numpy(a).to(dev).to(torch.bfloat16)  # noqa: E731
    # ---- packed [B, L, 3, H, D] buffer, views [B, H, L, D]
    w = workloads.make("packed", "bf16", 2, 3, 200, 64, 32, 3, 40, seed=22, lengths=(50, 200))
    qkv = torch.stack([bf(w.q), bf(w.k), bf(w.v)], dim=1)            # [B, 3, H, L, D]
    qkv = qkv.permute(0, 3, 1, 2, 4).contiguous().requires_grad_(True)   # [B, L, 3, H, D]
    q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    gate = torch.from_numpy(w.gate).to(dev).requires_grad_(True)
    lens = torch.from_numpy(w.seq_lens.astype(np.int64)).to(dev)
    guard = torch.full((1 << 20,), 7.0, device=dev)                  # a neighbour in the allocator's pool
    out, idx = blossom_attention(q, k, v, gate, w.block, w.topk, w.window, seq_lens=lens, return_indices=True)
    out.backward(bf(w.dout))
    torch.cuda.synchronize()
    assert bool((guard == 7.0).all())
    ref = oracle.forward_backward(w.q, w.k, w.v, w.gate, w.dout, w.block, w.topk, w.window, w.seq_lens,
                                  idx=idx.cpu().numpy())
    g = qkv.grad.permute(0, 2, 3, 1, 4)                              # [B, 3, H, L, D]
    got = {"out": out, "dq": g[:, 0], "dk": g[:, 1], "dv": g[:, 2], "dgate": gate.grad}
    for key, val in got.items():
        err = float(np.abs(val.detach().float().cpu().numpy() - ref[key]).max())
        assert err <= tolerance(w, ref[key]), (key, err)
    # ---- grouped heads
    w = workloads.make("autograd-gqa", "bf16", 2, 4, 256, 32, 32, 3, 48, seed=23, kv_heads=2)
    t = lambda a: bf(a).requires_grad_(True)  # noqa: E731
    q, k, v = t(w.q), t(w.k), t(w.v)
    gate = torch.from_numpy(w.gate).to(dev).requires_grad_(True)
    out, idx = blossom_attention(q, k, v, gate, w.block, w.topk, w.window, return_indices=True)
    out.backward(bf(w.dout))
    assert tuple(idx.shape) == (2, 2, 8, 3) and k.grad.shape == k.shape
    f = oracle.forward_gqa(w.q, w.k, w.v, w.gate, w.block, w.topk, w.window, idx=idx.cpu().numpy())
    ref = dict(f)
    ref.update(oracle.backward_gqa(w.q, w.k, w.v, w.gate, w.block, w.topk, w.window, f, w.dout))
    got = {"out": out, "dq": q.grad, "dk": k.grad, "dv": v.grad, "dgate": gate.grad}
    for key, val in got.items():
        err = float(np.abs(val.detach().float().cpu().numpy() - ref[key]).max())
        assert err <= tolerance(w, ref[key]), (key, err)


def test_autograd_options_input_dependent_gate_per_query_selection_learned_summary():
    """The front end's newer options together: Eq. 18's gate (gradient of F_o's parameters), a
    selection per query position, the learnable block summary."""
    import torch
    import oracle
    from paper_2512_13368_b200.autograd import blossom_attention
    dev = torch.device("cuda:0")
    w = workloads.make("autograd-opts", "fp32", 2, 2, 96, 32, 16, 3, 20, seed=71)
    gw = (0.3 * np.random.default_rng(1).standard_normal((2, 65))).astype(np.float32)
    phi = np.random.default_rng(2).standard_normal(16).astype(np.float32)
    t = lambda a: torch.from_numpy(a).to(dev).requires_grad_(True)  # noqa: E731
    q, k, v, gate = t(w.q), t(w.k), t(w.v), t(gw)
    out, idx = blossom_attention(q, k, v, gate, w.block, w.topk, w.window, return_indices=True,
                                 select_per_query=True, phi_logits=torch.from_numpy(phi).to(dev),
                                 input_dependent_gate=True)
    out.backward(torch.from_numpy(w.dout).to(dev))
    ref_idx = oracle.select_blocks_per_query(w.q, w.k, w.block, w.topk, phi_logits=phi)
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    ref = oracle.forward_backward(w.q, w.k, w.v, gw, w.dout, w.block, w.topk, w.window, idx=ref_idx,
                                  per_query=True, gate_mode=1)
    got = {"out": out, "dq": q.grad, "dk": k.grad, "dv": v.grad, "dgate": gate.grad}
    for key, val in got.items():
        err = float(np.abs(val.detach().float().cpu().numpy() - ref[key]).max())
        assert err <= 1e-4, (key, err)


def test_layer_step_runs_and_reports_attention_share():
    from paper_2512_13368_b200 import layer_step
    r = layer_step.attention_share(batch=8, seq_len=256, n_items=2000, negatives=15, steps=2, warmup=1)
    assert np.isfinite(r["loss"]) and r["loss"] > 0
    assert 0.0 < r["attention_share"] < 1.0
    assert r["library_launches_per_step"] >= 2 * 7   # two layers x (selection, forward, backward kernels)
