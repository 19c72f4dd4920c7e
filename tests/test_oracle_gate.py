"""Pins of the oracle's input-dependent gate (Eq. 18 with a one-layer F_o, Eq. 19): the reduction
to the scalar gate, a numpy evaluation of the forward from the branch outputs, central differences
for every input and for F_o's parameters, and PyTorch autograd through the dense-mask formula."""
import math

import numpy as np
import pytest

from oracle import blossom_oracle as oracle


def rand_case(seed, B=2, H=2, L=40, D=4):
    rng = np.random.default_rng(seed)
    q, k, v = (rng.standard_normal((B, H, L, D)) for _ in range(3))
    return q, k, v, 0.5 * rng.standard_normal((H, 2 * D + 1)), rng.standard_normal((B, H, L, D))


def test_zero_weights_are_the_scalar_gate():
    q, k, v, gw, dout = rand_case(1)
    D = 4
    g2 = np.random.default_rng(2).standard_normal((2, 2))
    gw[:] = 0.0
    gw[:, 2 * D] = g2[:, 0] - g2[:, 1]
    sl = np.asarray([40, 17], dtype=np.int32)
    a = oracle.forward_backward(q, k, v, g2, dout, 8, 3, 5, sl)
    b = oracle.forward_backward(q, k, v, gw, dout, 8, 3, 5, sl, gate_mode=1)
    for key in ("out", "out_lt", "out_st", "lse", "dq", "dk", "dv"):
        np.testing.assert_allclose(b[key], a[key], atol=1e-14)
    np.testing.assert_allclose(b["dgate"][:, 2 * D], a["dgate"][:, 0], atol=1e-12)   # d b = d a_lt


def test_forward_is_eq_18_and_19_on_the_branch_outputs():
    q, k, v, gw, dout = rand_case(3)
    D = 4
    f = oracle.forward(q, k, v, gw, 8, 3, 5, gate_mode=1)
    a = np.einsum("hd,bhld->bhl", gw[:, :D], f["out_lt"]) + np.einsum("hd,bhld->bhl", gw[:, D:2 * D], f["out_st"])
    alpha = 1.0 / (1.0 + np.exp(-(a + gw[None, :, None, 2 * D])))
    np.testing.assert_allclose(f["out"], alpha[..., None] * f["out_lt"] + (1 - alpha[..., None]) * f["out_st"], atol=1e-13)
    g0 = np.zeros((2, 2))
    f0 = oracle.forward(q, k, v, g0, 8, 3, 5, idx=f["idx"])
    np.testing.assert_array_equal(f0["out_lt"], f["out_lt"])       # the branches do not depend on the gate
    np.testing.assert_array_equal(f0["out_st"], f["out_st"])


@pytest.mark.parametrize("lens,per_query", [(None, False), ([40, 21], False), ([40, 21], True)])
def test_gradients_by_central_differences(lens, per_query):
    q, k, v, gw, dout = rand_case(4)
    sl = None if lens is None else np.asarray(lens, dtype=np.int32)
    f = oracle.forward(q, k, v, gw, 8, 3, 5, sl, gate_mode=1, per_query=per_query)
    g = oracle.backward(q, k, v, gw, 8, 3, 5, f, dout, sl, gate_mode=1, per_query=per_query)
    idx = f["idx"]

    def loss(q_, k_, v_, g_):
        return float((oracle.forward(q_, k_, v_, g_, 8, 3, 5, sl, idx=idx, gate_mode=1, per_query=per_query)["out"] * dout).sum())

    rng = np.random.default_rng(5)
    h = 1e-5
    arrs = [q, k, v, gw]
    for name, i in (("dq", 0), ("dk", 1), ("dv", 2), ("dgate", 3)):
        for _ in range(24):
            pos = tuple(int(rng.integers(0, n)) for n in arrs[i].shape)
            ap, am = arrs[i].copy(), arrs[i].copy()
            ap[pos] += h
            am[pos] -= h
            args_p, args_m = list(arrs), list(arrs)
            args_p[i], args_m[i] = ap, am
            fd = (loss(*args_p) - loss(*args_m)) / (2 * h)
            assert abs(fd - g[name][pos]) < 2e-7 * max(1.0, abs(fd)), (name, pos, fd, g[name][pos])


def test_autograd_through_the_dense_mask_formula():
    torch = pytest.importorskip("torch")
    L, Bk, topk, w, D = 32, 8, 2, 4, 4
    q, k, v, gw, dout = rand_case(6, B=1, H=1, L=L, D=D)
    f = oracle.forward(q, k, v, gw, Bk, topk, w, gate_mode=1)
    g = oracle.backward(q, k, v, gw, Bk, topk, w, f, dout, gate_mode=1)
    idx = f["idx"][0, 0]
    maskL = torch.zeros(L, L, dtype=torch.bool)
    maskS = torch.zeros(L, L, dtype=torch.bool)
    for t in range(L):
        for j in idx[t // Bk]:
            if j >= 0:
                maskL[t, j * Bk:min((j + 1) * Bk, t + 1)] = True
        maskS[t, max(0, t - w + 1):t + 1] = True
    tq, tk, tv, tg = (torch.tensor(a[0, 0] if a.ndim == 4 else a[0], dtype=torch.float64, requires_grad=True)
                      for a in (q, k, v, gw))
    s = (tq @ tk.T) / math.sqrt(D)
    oL = torch.softmax(s.masked_fill(~maskL, -math.inf), dim=1) @ tv
    oS = torch.softmax(s.masked_fill(~maskS, -math.inf), dim=1) @ tv
    alpha = torch.sigmoid(oL @ tg[:D] + oS @ tg[D:2 * D] + tg[2 * D])
    out = alpha[:, None] * oL + (1 - alpha[:, None]) * oS
    np.testing.assert_allclose(out.detach().numpy(), f["out"][0, 0], atol=1e-12)
    (out * torch.tensor(dout[0, 0])).sum().backward()
    np.testing.assert_allclose(tq.grad.numpy(), g["dq"][0, 0], atol=1e-11)
    np.testing.assert_allclose(tk.grad.numpy(), g["dk"][0, 0], atol=1e-11)
    np.testing.assert_allclose(tv.grad.numpy(), g["dv"][0, 0], atol=1e-11)
    np.testing.assert_allclose(tg.grad.numpy(), g["dgate"][0], atol=1e-11)
