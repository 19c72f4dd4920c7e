"""Pins of the oracle's selection per query position (Eq. 13 as the paper prints it) and of the
attention functions run on such a selection.

Independent of the oracle's code: blocks of one position (where the per-block and the per-position
selection are the same thing), queries repeated within a block, a numpy scorer with a stable
arg-sort, strict causality, an explicit dense-mask evaluation of Eq. 1 and central differences.
"""
import math

import numpy as np
import pytest

from oracle import blossom_oracle as oracle


def rand_case(seed, B=2, H=2, L=48, D=8, Hkv=None):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, H, L, D))
    k = rng.standard_normal((B, Hkv or H, L, D))
    v = rng.standard_normal((B, Hkv or H, L, D))
    return q, k, v, rng.standard_normal((H, 2)), rng.standard_normal((B, H, L, D))


def test_blocks_of_one_position_agree_with_the_per_block_selection():
    q, k, *_ = rand_case(1, L=40)
    sl = np.asarray([40, 23], dtype=np.int32)
    a = oracle.select_blocks(q, k, 1, 5, sl)
    b = oracle.select_blocks_per_query(q, k, 1, 5, sl)
    np.testing.assert_array_equal(a, b)


def test_equal_queries_in_a_block_select_what_the_block_selects():
    q, k, *_ = rand_case(2, L=64)
    q = np.repeat(q[:, :, ::8], 8, axis=2)           # every query of a block of 8 is the same vector
    per_block = oracle.select_blocks(q, k, 8, 3)
    per_query = oracle.select_blocks_per_query(q, k, 8, 3)
    np.testing.assert_array_equal(per_query, np.repeat(per_block, 8, axis=2))


@pytest.mark.parametrize("lens", [None, [50, 19]])
def test_against_a_numpy_scorer_with_stable_sort(lens):
    L, Bk, topk, D = 50, 8, 3, 8
    q, k, *_ = rand_case(3, L=L, D=D)
    sl = None if lens is None else np.asarray(lens, dtype=np.int32)
    idx, pr = oracle.select_blocks_per_query(q, k, Bk, topk, sl, return_scores=True)
    M = -(-L // Bk)
    for n in range(2):
        pad0 = 0 if sl is None else L - int(sl[n])
        for h in range(2):
            means, live = np.zeros((M, D)), np.zeros(M, dtype=bool)
            for j in range(M):
                lo, hi = max(j * Bk, pad0), min((j + 1) * Bk, L)
                if lo < hi:
                    means[j], live[j] = k[n, h, lo:hi].mean(axis=0), True
            for t in range(L):
                if t < pad0:
                    assert list(idx[n, h, t]) == [-1] * topk
                    continue
                b = t // Bk
                cand = [j for j in range(b) if live[j]]
                row = [b]
                if cand:
                    z = (q[n, h, t] @ means[cand].T) / math.sqrt(D)
                    p = np.exp(z - z.max())
                    p /= p.sum()
                    np.testing.assert_allclose(pr[n, h, t, cand], p, atol=1e-13)
                    assert abs(pr[n, h, t].sum() - 1.0) < 1e-12
                    order = np.argsort(-p, kind="stable")[:topk - 1]
                    row = sorted(int(cand[i]) for i in order) + [b]
                assert list(idx[n, h, t][:len(row)]) == row and all(x == -1 for x in idx[n, h, t][len(row):])


def test_exact_ties_go_to_the_lower_block():
    q, k, *_ = rand_case(4, B=1, H=1, L=64)
    k[:] = k[:, :, :1]                                # every block summary identical: all scores tie
    idx = oracle.select_blocks_per_query(q, k, 8, 3)
    for t in range(64):
        b = t // 8
        exp = list(range(min(b, 2))) + [b]
        assert list(idx[0, 0, t][:len(exp)]) == exp


def test_strictly_causal_selection_and_output():
    """Nothing at positions after t (not even later queries of t's own block) can change the
    selection of t or its output: the candidates of t are blocks that end before t's block."""
    q, k, v, gate, _ = rand_case(5, B=1, L=48)
    f0 = oracle.forward(q, k, v, gate, 8, 3, 5, per_query=True)
    rng = np.random.default_rng(0)
    for t in (3, 17, 30, 40):
        q2, k2, v2 = q.copy(), k.copy(), v.copy()
        q2[:, :, t + 1:] += rng.standard_normal(q2[:, :, t + 1:].shape)
        k2[:, :, t + 1:] += rng.standard_normal(k2[:, :, t + 1:].shape)
        v2[:, :, t + 1:] += rng.standard_normal(v2[:, :, t + 1:].shape)
        f1 = oracle.forward(q2, k2, v2, gate, 8, 3, 5, per_query=True)
        np.testing.assert_array_equal(f1["idx"][:, :, :t + 1], f0["idx"][:, :, :t + 1])
        np.testing.assert_array_equal(f1["out"][:, :, :t + 1], f0["out"][:, :, :t + 1])


def test_attention_on_a_per_position_selection_is_the_dense_mask_formula_and_its_gradient():
    L, Bk, topk, w, D = 40, 8, 3, 6, 4
    q, k, v, gate, dout = rand_case(6, B=1, H=2, L=L, D=D)
    sl = np.asarray([33], dtype=np.int32)
    pad0 = L - 33
    f = oracle.forward(q, k, v, gate, Bk, topk, w, sl, per_query=True)
    idx = f["idx"]
    scale = 1.0 / math.sqrt(D)
    for h in range(2):
        maskL = np.zeros((L, L), dtype=bool)
        maskS = np.zeros((L, L), dtype=bool)
        for t in range(pad0, L):
            for j in idx[0, h, t]:
                if j >= 0:
                    maskL[t, max(j * Bk, pad0):min((j + 1) * Bk, t + 1)] = True
            maskS[t, max(pad0, t - w + 1):t + 1] = True
        s = scale * q[0, h] @ k[0, h].T
        alpha = 1.0 / (1.0 + math.exp(-(gate[h, 0] - gate[h, 1])))
        outs = []
        for mask in (maskL, maskS):
            z = np.where(mask, s, -np.inf)
            with np.errstate(invalid="ignore"):
                p = np.exp(z - z.max(axis=1, keepdims=True))
            p = np.where(mask, p, 0.0)
            den = p.sum(axis=1, keepdims=True)
            outs.append(np.where(den > 0, p / np.where(den > 0, den, 1.0), 0.0) @ v[0, h])
        np.testing.assert_allclose(f["out_lt"][0, h], outs[0], atol=1e-12)
        np.testing.assert_allclose(f["out_st"][0, h], outs[1], atol=1e-12)
        np.testing.assert_allclose(f["out"][0, h], alpha * outs[0] + (1 - alpha) * outs[1], atol=1e-12)
    g = oracle.backward(q, k, v, gate, Bk, topk, w, f, dout, sl, per_query=True)

    def loss(q_, k_, v_):
        return float((oracle.forward(q_, k_, v_, gate, Bk, topk, w, sl, idx=idx, per_query=True)["out"] * dout).sum())

    rng = np.random.default_rng(1)
    hh = 1e-5
    for name, arr, i in (("dq", q, 0), ("dk", k, 1), ("dv", v, 2)):
        for _ in range(20):
            pos = tuple(int(rng.integers(0, n)) for n in arr.shape)
            args_p, args_m = [q, k, v], [q, k, v]
            ap, am = arr.copy(), arr.copy()
            ap[pos] += hh
            am[pos] -= hh
            args_p[i], args_m[i] = ap, am
            fd = (loss(*args_p) - loss(*args_m)) / (2 * hh)
            assert abs(fd - g[name][pos]) < 1e-7 * max(1.0, abs(fd)), (name, pos)


def test_grouped_heads_share_one_per_position_selection():
    q, k, v, gate, dout = rand_case(7, B=1, H=4, L=48, Hkv=2)
    idx, pr = oracle.select_blocks_per_query(q, k, 8, 3, return_scores=True)
    assert idx.shape == (1, 2, 48, 3)
    one = oracle.select_blocks_per_query(q[:, :2], k[:, :1], 8, 3, return_scores=True)[1]
    a = oracle.select_blocks_per_query(q[:, :1], k[:, :1], 8, 3, return_scores=True)[1]
    b = oracle.select_blocks_per_query(q[:, 1:2], k[:, :1], 8, 3, return_scores=True)[1]
    np.testing.assert_allclose(one[0, 0], a[0, 0] + b[0, 0], atol=1e-14)      # Eq. 12
    np.testing.assert_allclose(pr[0, 0], one[0, 0], atol=1e-14)
    f = oracle.forward_gqa(q, k, v, gate, 8, 3, 5, per_query=True)
    np.testing.assert_array_equal(f["idx"], idx)
    g = oracle.backward_gqa(q, k, v, gate, 8, 3, 5, f, dout, per_query=True)
    assert g["dk"].shape == k.shape


# ---- per position through overlapping compression blocks (Eq. 8-11, 13 as printed) ------------
def test_compression_blocks_equal_to_the_selection_blocks_change_nothing():
    q, k, *_ = rand_case(11, L=72)
    sl = np.asarray([72, 31], dtype=np.int32)
    a, pa = oracle.select_blocks_per_query(q, k, 8, 3, sl, return_scores=True)
    b, pb = oracle.select_blocks_per_query(q, k, 8, 3, sl, return_scores=True, cmp_block=8, cmp_stride=8)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_allclose(pa, pb, rtol=0, atol=1e-15)


def test_equal_queries_in_a_block_select_what_the_block_selects_through_compression_blocks():
    q, k, *_ = rand_case(12, L=96)
    q = np.repeat(q[:, :, ::8], 8, axis=2)           # every query of a block of 8 is the same vector
    per_block, sb, _ = oracle.select_blocks_cmp(q, k, 8, 3, 16, 4, return_scores=True)
    per_query, sq = oracle.select_blocks_per_query(q, k, 8, 3, return_scores=True, cmp_block=16, cmp_stride=4)
    np.testing.assert_array_equal(per_query, np.repeat(per_block, 8, axis=2))
    # a block's score is the sum over its 8 equal queries of the position's score
    np.testing.assert_allclose(np.repeat(sb, 8, axis=2), 8.0 * sq, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("lens", [None, [70, 27]])
@pytest.mark.parametrize("Bk,l,s", [(8, 16, 4), (16, 32, 16), (8, 8, 4)])
def test_compression_blocks_against_a_numpy_scorer(lens, Bk, l, s):
    """Means by slicing, one softmax per position over the compression blocks that end before the
    position's block, Eq. 11 as a double sum, stable arg-sort: written without the oracle's code."""
    L, topk, D = 70, 3, 8
    q, k, *_ = rand_case(13, L=L, D=D)
    sl = None if lens is None else np.asarray(lens, dtype=np.int32)
    idx, sc = oracle.select_blocks_per_query(q, k, Bk, topk, sl, return_scores=True, cmp_block=l, cmp_stride=s)
    M, Mc = -(-L // Bk), (L - l) // s + 1
    for n in range(2):
        pad0 = 0 if sl is None else L - int(sl[n])
        for h in range(2):
            means, live = np.zeros((Mc, D)), np.zeros(Mc, dtype=bool)
            for i in range(Mc):
                lo = max(i * s, pad0)
                if lo < i * s + l:
                    means[i], live[i] = k[n, h, lo:i * s + l].mean(axis=0), True
            for t in range(L):
                if t < pad0:
                    assert list(idx[n, h, t]) == [-1] * topk
                    continue
                b = t // Bk
                cands = [i for i in range(Mc) if i * s + l <= b * Bk and live[i]]
                p = np.zeros(Mc)
                if cands:
                    z = (means[cands] @ q[n, h, t]) / math.sqrt(D)
                    e = np.exp(z - z.max())
                    p[cands] = e / e.sum()
                S = np.zeros(M)
                for j in range(b):
                    for m in range(Bk // s):
                        for r in range(l // s):
                            i = (Bk // s) * j - m - r
                            if 0 <= i < Mc and i * s + l <= b * Bk:
                                S[j] += p[i]
                sel = [j for j in range(b) if min((j + 1) * Bk, L) > max(j * Bk, pad0)]
                order = sorted(sel, key=lambda j: (-S[j], j))[:topk - 1]
                want = sorted(order) + [b]
                assert [int(x) for x in idx[n, h, t] if x >= 0] == want, (n, h, t)
                np.testing.assert_allclose(sc[n, h, t, sel], S[sel], rtol=1e-12, atol=1e-14)


def test_grouped_heads_sum_the_mapped_probabilities_of_a_position():
    q, k, *_ = rand_case(14, H=4, Hkv=2, L=64)
    idx, sc = oracle.select_blocks_per_query(q, k, 8, 3, return_scores=True, cmp_block=16, cmp_stride=8)
    assert idx.shape == (2, 2, 64, 3)
    _, per_head = oracle.select_blocks_per_query(q, np.repeat(k, 2, axis=1), 8, 3, return_scores=True,
                                                 cmp_block=16, cmp_stride=8)
    np.testing.assert_allclose(sc, per_head.reshape(2, 2, 2, 64, 8).sum(axis=2), rtol=1e-13, atol=1e-15)
    t = 63
    row = [int(x) for x in idx[0, 1, t] if x >= 0]
    best = sorted(range(7), key=lambda j: (-sc[0, 1, t, j], j))[:2]
    assert row == sorted(best) + [7]
