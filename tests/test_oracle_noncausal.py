"""Pins of the oracle without the causal mask (the bidirectional encoders the paper also plugs the
mechanism into): reductions to dense bidirectional attention (a library routine), the dense-mask
formula with the symmetric Eq. 15, a numpy scorer for the selection, central differences."""
import math

import numpy as np
import pytest

from oracle import blossom_oracle as oracle


def rand_case(seed, B=2, H=2, L=40, D=4):
    rng = np.random.default_rng(seed)
    q, k, v = (rng.standard_normal((B, H, L, D)) for _ in range(3))
    return q, k, v, rng.standard_normal((H, 2)), rng.standard_normal((B, H, L, D))


def test_everything_visible_is_dense_bidirectional_attention():
    torch = pytest.importorskip("torch")
    q, k, v, gate, _ = rand_case(1)
    f = oracle.forward(q, k, v, gate, 8, 5, 40, causal=False)        # top-k = all blocks, window >= L
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.tensor(q), torch.tensor(k), torch.tensor(v), is_causal=False).numpy()
    for key in ("out", "out_lt", "out_st"):
        np.testing.assert_allclose(f[key], ref, atol=1e-12)


@pytest.mark.parametrize("mode,blk", [(0, 1), (1, 1), (1, 4)])
def test_dense_mask_formula_with_the_symmetric_short_term_mask(mode, blk):
    L, Bk, topk, w, D = 40, 8, 3, 3, 4
    q, k, v, gate, _ = rand_case(2, B=1, L=L, D=D)
    sl = np.asarray([31], dtype=np.int32)
    pad0 = L - 31
    f = oracle.forward(q, k, v, gate, Bk, topk, w, sl, stis_mode=mode, stis_block=blk, causal=False)
    for h in range(2):
        mL = np.zeros((L, L), dtype=bool)
        mS = np.zeros((L, L), dtype=bool)
        for t in range(pad0, L):
            for j in f["idx"][0, h, t // Bk]:
                if j >= 0:
                    mL[t, max(j * Bk, pad0):min((j + 1) * Bk, L)] = True
            for p in range(pad0, L):
                d = abs(t // blk - p // blk)
                mS[t, p] = abs(t - p) < w or (mode == 1 and ((d >= 1 and d & (d - 1) == 0) or p >= L - blk))
        s = q[0, h] @ k[0, h].T / math.sqrt(D)
        for mask, key in ((mL, "out_lt"), (mS, "out_st")):
            z = np.where(mask, s, -np.inf)
            with np.errstate(invalid="ignore"):
                p_ = np.where(mask, np.exp(z - z.max(axis=1, keepdims=True)), 0.0)
            den = p_.sum(axis=1, keepdims=True)
            o = np.where(den > 0, p_ / np.where(den > 0, den, 1.0), 0.0) @ v[0, h]
            np.testing.assert_allclose(f[key][0, h], o, atol=1e-12)
        assert mS[pad0 + 5].sum() > (2 * w - 1 if mode else 0) - 1       # keys on both sides


def test_selection_scores_every_other_live_block():
    L, Bk, topk, D = 48, 8, 3, 4
    q, k, *_ = rand_case(3, L=L, D=D)
    sl = np.asarray([48, 21], dtype=np.int32)
    idx, sc = oracle.select_blocks(q, k, Bk, topk, sl, return_scores=True, causal=False)
    M = L // Bk
    for n in range(2):
        pad0 = L - int(sl[n])
        for h in range(2):
            live = [(j + 1) * Bk > pad0 for j in range(M)]
            means = np.array([k[n, h, max(j * Bk, pad0):(j + 1) * Bk].mean(axis=0) if live[j] else np.zeros(D)
                              for j in range(M)])
            for b in range(M):
                if not live[b]:
                    assert list(idx[n, h, b]) == [-1] * topk
                    continue
                cand = [j for j in range(M) if live[j] and j != b]
                z = q[n, h, max(b * Bk, pad0):(b + 1) * Bk] @ means[cand].T / math.sqrt(D)
                p = np.exp(z - z.max(axis=1, keepdims=True))
                S = (p / p.sum(axis=1, keepdims=True)).sum(axis=0)
                np.testing.assert_allclose(sc[n, h, b, cand], S, atol=1e-12)
                best = sorted(cand, key=lambda j: (-S[cand.index(j)], j))[:topk - 1]
                row = sorted(best + [b])
                assert list(idx[n, h, b][:len(row)]) == row


def test_gradients_by_central_differences():
    q, k, v, gate, dout = rand_case(4)
    sl = np.asarray([40, 26], dtype=np.int32)
    f = oracle.forward(q, k, v, gate, 8, 3, 4, sl, stis_mode=1, causal=False)
    g = oracle.backward(q, k, v, gate, 8, 3, 4, f, dout, sl, stis_mode=1, causal=False)
    idx = f["idx"]

    def loss(q_, k_, v_, g_):
        return float((oracle.forward(q_, k_, v_, g_, 8, 3, 4, sl, idx=idx, stis_mode=1, causal=False)["out"] * dout).sum())

    rng = np.random.default_rng(5)
    h = 1e-5
    arrs = [q, k, v, gate]
    for name, i in (("dq", 0), ("dk", 1), ("dv", 2), ("dgate", 3)):
        for _ in range(20):
            pos = tuple(int(rng.integers(0, n)) for n in arrs[i].shape)
            ap, am = arrs[i].copy(), arrs[i].copy()
            ap[pos] += h
            am[pos] -= h
            a_p, a_m = list(arrs), list(arrs)
            a_p[i], a_m[i] = ap, am
            fd = (loss(*a_p) - loss(*a_m)) / (2 * h)
            assert abs(fd - g[name][pos]) < 2e-7 * max(1.0, abs(fd)), (name, pos)
