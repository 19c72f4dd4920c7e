"""Pins for the fp64 CPU oracle: it is checked against things other than itself.

  P1  explicit dense 0/1 masks + the masked-softmax definition (Eq. 1) in numpy
  P2  invariants (index structure, causality, softmax rows)
  P3  reductions to textbook dense causal attention (torch's SDPA on CPU, fp64)
  P4  constructed selections whose answer is known by construction (incl. exact ties)
  P5  a second, independently written scorer + stable sort
  P6  finite differences and torch autograd through the dense-mask formula
  P7  Table 5's printed key budgets (tests/golden/table5_participation.txt)
  P8  permutation / linearity / gate-shift equivariances
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_case(seed, B=2, H=2, L=37, D=8, lens=None):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, H, L, D))
    k = rng.standard_normal((B, H, L, D))
    v = rng.standard_normal((B, H, L, D))
    gate = rng.standard_normal((H, 2))
    dout = rng.standard_normal((B, H, L, D))
    sl = None
    if lens is not None:
        sl = np.asarray(lens, dtype=np.int32)
    return q, k, v, gate, dout, sl


# --------------------------------------------------------------------------- P1
def dense_masks(idx, L, block, window, seq_lens):
    """0/1 masks [B,H,L,L] of the two branches, written from the definitions."""
    B, H, M, K = idx.shape
    mL = np.zeros((B, H, L, L), dtype=bool)
    mS = np.zeros((B, H, L, L), dtype=bool)
    t = np.arange(L)[:, None]
    p = np.arange(L)[None, :]
    causal = p <= t
    win = (t - p) < window
    for n in range(B):
        pad0 = 0 if seq_lens is None else L - int(seq_lens[n])
        valid = (t >= pad0) & (p >= pad0)
        for h in range(H):
            sel = np.zeros((L, L), dtype=bool)
            for b in range(M):
                rows = slice(b * block, min((b + 1) * block, L))
                for j in idx[n, h, b]:
                    if j >= 0:
                        sel[rows, j * block:min((j + 1) * block, L)] = True
            mL[n, h] = sel & causal & valid
            mS[n, h] = win & causal & valid
    return mL, mS


def masked_attention(q, k, v, mask, scale):
    """softmax(scale QK^T + log M) V with rows of an all-zero mask giving 0; also returns lse."""
    s = np.einsum("bhtd,bhpd->bhtp", q, k) * scale
    s = np.where(mask, s, -np.inf)
    mx = np.max(s, axis=-1, keepdims=True)
    mx = np.where(np.isfinite(mx), mx, 0.0)
    e = np.exp(s - mx)
    den = e.sum(-1, keepdims=True)
    any_ = mask.any(-1, keepdims=True)
    p = np.where(any_, e / np.where(any_, den, 1.0), 0.0)
    lse = np.where(any_[..., 0], mx[..., 0] + np.log(np.where(any_, den, 1.0))[..., 0], 0.0)
    return np.einsum("bhtp,bhpd->bhtd", p, v), lse, p


@pytest.mark.parametrize("L,block,topk,window,lens", [
    (37, 8, 3, 5, None),
    (64, 8, 2, 16, None),
    (50, 16, 4, 32, [50, 5]),
    (40, 4, 5, 9, [17, 40]),
    (33, 8, 1, 1, [33, 1]),
])
def test_p1_dense_mask_definition(L, block, topk, window, lens):
    q, k, v, gate, dout, sl = rand_case(1, L=L, lens=lens)
    D = q.shape[-1]
    f = oracle.forward(q, k, v, gate, block, topk, window, sl)
    mL, mS = dense_masks(f["idx"], L, block, window, sl)
    scale = 1.0 / math.sqrt(D)
    oL, lL, pL = masked_attention(q, k, v, mL, scale)
    oS, lS, pS = masked_attention(q, k, v, mS, scale)
    np.testing.assert_allclose(f["out_lt"], oL, atol=1e-12)
    np.testing.assert_allclose(f["out_st"], oS, atol=1e-12)
    np.testing.assert_allclose(f["lse"][0], lL, atol=1e-12)
    np.testing.assert_allclose(f["lse"][1], lS, atol=1e-12)
    alpha = 1.0 / (1.0 + np.exp(-(gate[:, 0] - gate[:, 1])))
    a = alpha[None, :, None, None]
    np.testing.assert_allclose(f["out"], a * oL + (1 - a) * oS, atol=1e-12)
    # softmax rows of valid queries sum to one in both branches
    B = q.shape[0]
    for n in range(B):
        pad0 = 0 if sl is None else L - int(sl[n])
        np.testing.assert_allclose(pL[n, :, pad0:].sum(-1), 1.0, atol=1e-12)
        np.testing.assert_allclose(pS[n, :, pad0:].sum(-1), 1.0, atol=1e-12)
        assert np.all(f["out"][n, :, :pad0] == 0.0)
        assert np.all(f["lse"][:, n, :, :pad0] == 0.0)


# --------------------------------------------------------------------------- P2
@pytest.mark.parametrize("lens", [None, [29, 7, 41]])
def test_p2_index_structure(lens):
    L, block, topk = 41, 4, 4
    q, k, v, gate, dout, sl = rand_case(2, B=3, L=L, lens=lens)
    idx = oracle.select_blocks(q, k, block, topk, sl)
    B, H, M, K = idx.shape
    assert (M, K) == (11, topk)
    for n in range(B):
        pad0 = 0 if sl is None else L - int(sl[n])
        live = [min((j + 1) * block, L) > max(j * block, pad0) for j in range(M)]
        for h in range(H):
            for b in range(M):
                row = idx[n, h, b]
                got = [int(j) for j in row if j >= 0]
                if not live[b]:
                    assert got == []
                    continue
                ncand = sum(live[:b])
                assert len(got) == min(topk, 1 + ncand)
                assert got == sorted(set(got)) and got[-1] == b
                assert all(live[j] for j in got)
                assert list(row[len(got):]) == [-1] * (K - len(got))


def test_p2_causality():
    L, block, topk, window = 48, 8, 3, 10
    q, k, v, gate, dout, sl = rand_case(3, L=L)
    f0 = oracle.forward(q, k, v, gate, block, topk, window)
    rng = np.random.default_rng(0)
    t0 = 21
    # (a) frozen selection: nothing after t0 influences rows <= t0
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[:, :, t0 + 1:] += rng.standard_normal(q2[:, :, t0 + 1:].shape)
    k2[:, :, t0 + 1:] += rng.standard_normal(k2[:, :, t0 + 1:].shape)
    v2[:, :, t0 + 1:] += rng.standard_normal(v2[:, :, t0 + 1:].shape)
    f1 = oracle.forward(q2, k2, v2, gate, block, topk, window, idx=f0["idx"])
    for key in ("out", "out_lt", "out_st"):
        assert np.array_equal(f0[key][:, :, :t0 + 1], f1[key][:, :, :t0 + 1])
    assert np.array_equal(f0["lse"][:, :, :, :t0 + 1], f1["lse"][:, :, :, :t0 + 1])
    # (b) live selection: later BLOCKS influence neither the indices nor the outputs of earlier blocks
    b0 = 3
    e = b0 * block
    q3, k3, v3 = q.copy(), k.copy(), v.copy()
    q3[:, :, e:] += rng.standard_normal(q3[:, :, e:].shape)
    k3[:, :, e:] += rng.standard_normal(k3[:, :, e:].shape)
    v3[:, :, e:] += rng.standard_normal(v3[:, :, e:].shape)
    f2 = oracle.forward(q3, k3, v3, gate, block, topk, window)
    assert np.array_equal(f0["idx"][:, :, :b0], f2["idx"][:, :, :b0])
    assert np.array_equal(f0["out"][:, :, :e], f2["out"][:, :, :e])


# --------------------------------------------------------------------------- P3
def sdpa_causal(q, k, v):
    tq, tk, tv = (torch.from_numpy(x) for x in (q, k, v))
    return torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).numpy()


def test_p3_reduces_to_dense_causal_attention():
    L, block = 40, 8
    q, k, v, gate, dout, sl = rand_case(4, L=L)
    dense = sdpa_causal(q, k, v)
    M = 5
    # window = L  => short-term branch is dense; top-k >= M => long-term branch is dense
    f = oracle.forward(q, k, v, gate, block, M, L)
    np.testing.assert_allclose(f["out_st"], dense, atol=1e-12)
    np.testing.assert_allclose(f["out_lt"], dense, atol=1e-12)
    np.testing.assert_allclose(f["out"], dense, atol=1e-12)          # for every gate
    f = oracle.forward(q, k, v, gate, block, M + 3, L + 5)           # larger than needed
    np.testing.assert_allclose(f["out"], dense, atol=1e-12)
    # each alone
    f = oracle.forward(q, k, v, gate, block, 2, L)
    np.testing.assert_allclose(f["out_st"], dense, atol=1e-12)
    assert np.abs(f["out_lt"] - dense).max() > 1e-3
    f = oracle.forward(q, k, v, gate, block, M, 3)
    np.testing.assert_allclose(f["out_lt"], dense, atol=1e-12)
    assert np.abs(f["out_st"] - dense).max() > 1e-3


def test_p3_block_diagonal_window_one_and_gate_limits():
    L, block = 40, 8
    q, k, v, gate, dout, sl = rand_case(5, L=L)
    f = oracle.forward(q, k, v, gate, block, 1, 1)
    # top-k = 1: only the own block -> dense causal attention inside each block
    for b in range(L // block):
        s = slice(b * block, (b + 1) * block)
        np.testing.assert_allclose(f["out_lt"][:, :, s], sdpa_causal(q[:, :, s], k[:, :, s], v[:, :, s]),
                                   atol=1e-12)
    # window = 1: the query sees itself only
    np.testing.assert_allclose(f["out_st"], v, atol=1e-14)
    np.testing.assert_allclose(f["lse"][1], np.einsum("bhtd,bhtd->bht", q, k) / math.sqrt(q.shape[-1]),
                               atol=1e-12)
    # gate limits: equal logits -> mean; +-40 -> one branch (the single-branch ablation variants)
    g = np.array([[0.3, 0.3], [-1.0, -1.0]])
    f = oracle.forward(q, k, v, g, block, 3, 6)
    np.testing.assert_allclose(f["out"], 0.5 * (f["out_lt"] + f["out_st"]), atol=1e-14)
    g = np.array([[40.0, 0.0], [0.0, 40.0]])
    f = oracle.forward(q, k, v, g, block, 3, 6)
    np.testing.assert_allclose(f["out"][:, 0], f["out_lt"][:, 0], atol=1e-14)
    np.testing.assert_allclose(f["out"][:, 1], f["out_st"][:, 1], atol=1e-14)


# --------------------------------------------------------------------------- P4
def constructed(c, block, D=8, seed=0):
    """keys constant inside block j: k_p = c[j] * u; all queries = u  =>  block logits rank like c."""
    rng = np.random.default_rng(seed)
    u = rng.standard_normal(D)
    M = len(c)
    L = M * block
    k = np.repeat(np.asarray(c, dtype=np.float64), block)[:, None] * u[None, :]
    q = np.tile(u, (L, 1))
    return q[None, None], k[None, None]


def test_p4_constructed_ranking_and_ties():
    block, topk = 4, 4
    c = [0.5, 2.0, -1.0, 1.5, 0.1, 3.0, 0.0, 0.7]
    q, k = constructed(c, block)
    idx = oracle.select_blocks(q, k, block, topk)[0, 0]
    for b in range(len(c)):
        past = sorted(range(b), key=lambda j: (-c[j], j))[:topk - 1]
        exp = sorted(past) + [b]
        assert [int(x) for x in idx[b] if x >= 0] == exp, (b, idx[b], exp)
    # exact ties: equal summaries give bit-identical scores; the lower index must win
    c = [1.0, 1.0, 1.0, 0.0, 1.0, 1.0, 2.0, 1.0]
    q, k = constructed(c, block)
    idx = oracle.select_blocks(q, k, block, 3)[0, 0]
    assert list(idx[3]) == [0, 1, 3]
    assert list(idx[5]) == [0, 1, 5]
    assert list(idx[7]) == [0, 6, 7]
    # a sign error in the logits or a "smallest-k" bug would pick block 3 (c = 0) here
    assert 3 not in idx[6]


def test_p4_single_valid_query_uses_raw_logits():
    # one valid query in the last block => its selection is the top-(k-1) of the raw logits
    rng = np.random.default_rng(7)
    L, block, D, topk = 33, 8, 8, 3
    q = rng.standard_normal((1, 1, L, D))
    k = rng.standard_normal((1, 1, L, D))
    idx = oracle.select_blocks(q, k, block, topk)[0, 0]
    ktil = np.stack([k[0, 0, j * block:(j + 1) * block].mean(0) for j in range(4)])
    z = ktil @ q[0, 0, 32]
    exp = sorted(np.argsort(-z)[:topk - 1].tolist()) + [4]
    assert list(idx[4]) == exp


# --------------------------------------------------------------------------- P5
def scorer_numpy(q, k, block, topk, seq_lens, scale):
    """Second implementation: matrix form + stable argsort on (-score, index)."""
    B, H, L, D = q.shape
    M = -(-L // block)
    out = -np.ones((B, H, M, topk), dtype=np.int32)
    S_all = np.zeros((B, H, M, M))
    for n in range(B):
        pad0 = 0 if seq_lens is None else L - int(seq_lens[n])
        valid = np.arange(L) >= pad0
        blk = np.arange(L) // block
        onehot = (blk[None, :] == np.arange(M)[:, None]) & valid[None, :]      # [M, L]
        cnt = onehot.sum(1)
        live = cnt > 0
        for h in range(H):
            ktil = (onehot.astype(np.float64) @ k[n, h]) / np.maximum(cnt, 1)[:, None]
            z = (q[n, h] @ ktil.T) * scale                                    # [L, M]
            for b in range(M):
                if not live[b]:
                    continue
                cand = np.flatnonzero(live[:b])
                rows = np.flatnonzero(onehot[b])
                pick = []
                if len(cand):
                    zz = z[np.ix_(rows, cand)]
                    pr = np.exp(zz - zz.max(1, keepdims=True))
                    pr /= pr.sum(1, keepdims=True)
                    S = pr.sum(0)
                    S_all[n, h, b, cand] = S
                    order = np.argsort(-S, kind="stable")
                    pick = cand[order[:topk - 1]].tolist()
                res = sorted(pick) + [b]
                out[n, h, b, :len(res)] = res
    return out, S_all


@pytest.mark.parametrize("lens", [None, [60, 9, 33]])
def test_p5_independent_scorer(lens):
    L, block, topk, D = 60, 4, 5, 8
    q, k, v, gate, dout, sl = rand_case(8, B=3, L=L, D=D, lens=lens)
    idx, S = oracle.select_blocks(q, k, block, topk, sl, return_scores=True)
    idx2, S2 = scorer_numpy(q, k, block, topk, sl, 1.0 / math.sqrt(D))
    np.testing.assert_allclose(S, S2, atol=1e-12)
    assert np.array_equal(idx, idx2)
    # non-default scale changes block-summed scores; check it is honoured
    idx3, S3 = oracle.select_blocks(q, k, block, topk, sl, sm_scale=1.7, return_scores=True)
    idx4, S4 = scorer_numpy(q, k, block, topk, sl, 1.7)
    np.testing.assert_allclose(S3, S4, atol=1e-12)
    assert np.array_equal(idx3, idx4)


# --------------------------------------------------------------------------- P6
def loss_np(q, k, v, gate, dout, block, topk, window, sl, idx):
    return float((oracle.forward(q, k, v, gate, block, topk, window, sl, idx=idx)["out"] * dout).sum())


@pytest.mark.parametrize("lens", [None, [26, 11]])
def test_p6_finite_differences(lens):
    L, block, topk, window = 26, 4, 3, 6
    q, k, v, gate, dout, sl = rand_case(9, L=L, D=4, lens=lens)
    r = oracle.forward_backward(q, k, v, gate, dout, block, topk, window, sl)
    idx = r["idx"]
    h = 1e-5
    rng = np.random.default_rng(1)
    for name, arr in (("dq", q), ("dk", k), ("dv", v), ("dgate", gate)):
        flat = arr.reshape(-1)
        picks = rng.choice(flat.size, size=min(flat.size, 160), replace=False)
        for i in picks:
            old = flat[i]
            flat[i] = old + h
            lp = loss_np(q, k, v, gate, dout, block, topk, window, sl, idx)
            flat[i] = old - h
            lm = loss_np(q, k, v, gate, dout, block, topk, window, sl, idx)
            flat[i] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - r[name].reshape(-1)[i]) < 1e-7 * max(1.0, abs(fd)), (name, i, fd)
    # padded rows receive and emit zero gradient
    if sl is not None:
        for n in range(q.shape[0]):
            pad0 = L - int(sl[n])
            for name in ("dq", "dk", "dv"):
                assert np.all(r[name][n, :, :pad0] == 0.0)


def test_p6_autograd_through_dense_mask_formula():
    L, block, topk, window = 30, 8, 3, 7
    q, k, v, gate, dout, sl = rand_case(10, L=L, D=8, lens=[30, 13])
    r = oracle.forward_backward(q, k, v, gate, dout, block, topk, window, sl)
    mL, mS = dense_masks(r["idx"], L, block, window, sl)
    tq, tk, tv, tg = (torch.tensor(x, requires_grad=True) for x in (q, k, v, gate))
    rowvalid = torch.tensor(mS.any(-1))

    def branch(mask):
        s = torch.einsum("bhtd,bhpd->bhtp", tq, tk) / math.sqrt(q.shape[-1])
        s = s.masked_fill(~torch.tensor(mask), float("-inf"))
        s = torch.where(rowvalid[..., None], s, torch.zeros_like(s))
        p = torch.softmax(s, -1)
        p = torch.where(rowvalid[..., None], p, torch.zeros_like(p))
        return torch.einsum("bhtp,bhpd->bhtd", p, tv)

    alpha = torch.sigmoid(tg[:, 0] - tg[:, 1])[None, :, None, None]
    out = alpha * branch(mL) + (1 - alpha) * branch(mS)
    (out * torch.tensor(dout)).sum().backward()
    np.testing.assert_allclose(r["dq"], tq.grad.numpy(), atol=1e-11)
    np.testing.assert_allclose(r["dk"], tk.grad.numpy(), atol=1e-11)
    np.testing.assert_allclose(r["dv"], tv.grad.numpy(), atol=1e-11)
    np.testing.assert_allclose(r["dgate"], tg.grad.numpy(), atol=1e-11)


# --------------------------------------------------------------------------- P7
def test_p7_table5_key_budget():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "table5_participation.txt"))
            if ln.strip() and not ln.startswith("#")]
    stride, sel_block, n_sel, win = 16, 16, 4, 8
    for L, full, blossom, red in rows:
        L, full, blossom, red = int(L), int(full), int(blossom), float(red)
        # the printed counts decompose as: scored blocks + selected keys + symmetric strict
        # window + power-of-two links
        assert blossom == L // stride + n_sel * sel_block + (2 * win - 1) + int(math.log2(L))
        assert abs(100.0 * (1 - blossom / full) - red) < 0.06
    # The oracle's masks realise the two terms on this path: with q = 0 every visible key has
    # the same weight, so exp(lse) counts the keys of a row.
    L, D = 256, 4
    rng = np.random.default_rng(0)
    q = np.zeros((1, 1, L, D))
    k = rng.standard_normal((1, 1, L, D))
    v = rng.standard_normal((1, 1, L, D))
    f = oracle.forward(q, k, v, np.zeros((1, 2)), sel_block, n_sel, win)
    nL = np.exp(f["lse"][0, 0, 0])
    nS = np.exp(f["lse"][1, 0, 0])
    t = np.arange(L)
    # selected keys: (n_sel - 1) full past blocks + the causal part of the own block
    full_rows = t >= (n_sel - 1) * sel_block
    np.testing.assert_allclose(nL[full_rows], ((n_sel - 1) * sel_block + t % sel_block + 1)[full_rows],
                               rtol=1e-12)
    last_rows = full_rows & (t % sel_block == sel_block - 1)
    np.testing.assert_allclose(nL[last_rows], n_sel * sel_block, rtol=1e-12)     # the 4*16 term
    # window: |i-j| < win, causal side -> win keys including the query itself ((2*win-1+1)/2)
    np.testing.assert_allclose(nS[t >= win - 1], win, rtol=1e-12)
    np.testing.assert_allclose(nS[t < win - 1], (t + 1)[t < win - 1], rtol=1e-12)
    assert np.all(nL <= n_sel * sel_block + 1e-9) and np.all(nS <= win + 1e-9)


# --------------------------------------------------------------------------- P8
def test_p8_equivariances():
    L, block, topk, window = 32, 8, 3, 5
    q, k, v, gate, dout, sl = rand_case(11, B=3, H=2, L=L, lens=[32, 20, 3])
    r = oracle.forward_backward(q, k, v, gate, dout, block, topk, window, sl)
    # permute batch entries and heads
    pb, ph = [2, 0, 1], [1, 0]
    r2 = oracle.forward_backward(q[pb][:, ph], k[pb][:, ph], v[pb][:, ph], gate[ph], dout[pb][:, ph],
                                 block, topk, window, sl[pb])
    for key in ("out", "out_lt", "out_st", "dq", "dk", "dv"):
        np.testing.assert_allclose(r[key][pb][:, ph], r2[key], atol=1e-13)
    assert np.array_equal(r["idx"][pb][:, ph], r2["idx"])
    np.testing.assert_allclose(r["dgate"][ph], r2["dgate"], atol=1e-12)
    # linear in v
    f3 = oracle.forward(q, k, 2.5 * v, gate, block, topk, window, sl)
    np.testing.assert_allclose(f3["out"], 2.5 * r["out"], atol=1e-12)
    # adding a constant to both gate logits changes nothing
    f4 = oracle.forward(q, k, v, gate + 3.25, block, topk, window, sl)
    np.testing.assert_allclose(f4["out"], r["out"], atol=1e-14)
    # dgate columns are opposite (alpha depends on the logit difference only)
    np.testing.assert_allclose(r["dgate"][:, 0], -r["dgate"][:, 1], atol=0)


def test_config1_oracle_runs_in_seconds():
    from paper_2512_13368_b200 import workloads
    w = workloads.config1()
    r = oracle.forward_backward(w.q, w.k, w.v, w.gate, w.dout, w.block, w.topk, w.window)
    assert r["out"].shape == (4, 2, 64, 32) and np.isfinite(r["dq"]).all()
    assert r["idx"].shape == (4, 2, 8, 2)
