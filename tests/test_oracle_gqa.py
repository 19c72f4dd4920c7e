"""Pins of the oracle's grouped-query functions (heads of a KV group share K, V and one selection
made from their summed scores, Eq. 12)."""
import math

import numpy as np
import pytest

from oracle import blossom_oracle as oracle


def rand_case(seed, B=2, H=4, Hkv=2, L=48, D=8, lens=None):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, H, L, D))
    k = rng.standard_normal((B, Hkv, L, D))
    v = rng.standard_normal((B, Hkv, L, D))
    gate = rng.standard_normal((H, 2))
    dout = rng.standard_normal((B, H, L, D))
    sl = None if lens is None else np.asarray(lens, dtype=np.int32)
    return q, k, v, gate, dout, sl


def test_one_head_per_group_is_ordinary_multi_head_attention():
    q, k, v, gate, dout, sl = rand_case(1, H=3, Hkv=3, lens=[48, 17])
    idx, sc = oracle.select_blocks_gqa(q, k, 8, 3, sl, return_scores=True)
    idx0, sc0 = oracle.select_blocks(q, k, 8, 3, sl, return_scores=True)
    np.testing.assert_array_equal(idx, idx0)
    np.testing.assert_array_equal(sc, sc0)
    f = oracle.forward_gqa(q, k, v, gate, 8, 3, 6, sl)
    f0 = oracle.forward(q, k, v, gate, 8, 3, 6, sl)
    for key in ("out", "out_lt", "out_st", "lse"):
        np.testing.assert_array_equal(f[key], f0[key])
    b = oracle.backward_gqa(q, k, v, gate, 8, 3, 6, f, dout, sl)
    b0 = oracle.backward(q, k, v, gate, 8, 3, 6, f0, dout, sl)
    for key in ("dq", "dk", "dv", "dgate"):
        np.testing.assert_array_equal(b[key], b0[key])


def test_group_scores_are_the_sum_of_an_independent_per_head_scorer():
    """Eq. 12 on a case small enough to score with plain numpy: block means, per-query softmax
    over the strictly-past blocks, sum over the block's queries and over the group's heads."""
    q, k, v, gate, dout, sl = rand_case(2, B=1, H=4, Hkv=2, L=32, D=4)
    blk, M, scale = 8, 4, 1.0 / math.sqrt(4)
    idx, sc = oracle.select_blocks_gqa(q, k, blk, 2, return_scores=True)
    for g in range(2):
        means = k[0, g].reshape(M, blk, 4).mean(axis=1)
        for b in range(1, M):
            s = np.zeros(b)
            for h in (2 * g, 2 * g + 1):
                z = scale * q[0, h, b * blk:(b + 1) * blk] @ means[:b].T
                p = np.exp(z - z.max(axis=1, keepdims=True))
                s += (p / p.sum(axis=1, keepdims=True)).sum(axis=0)
            np.testing.assert_allclose(sc[0, g, b, :b], s, atol=1e-12)
            assert list(idx[0, g, b]) == sorted([int(np.argmax(s)), b])   # top-1 past block + own block


def test_identical_heads_in_a_group_select_like_one_head():
    q, k, v, gate, dout, sl = rand_case(3, H=2, Hkv=1, lens=[48, 30])
    q[:, 1] = q[:, 0]
    idx = oracle.select_blocks_gqa(q, k, 8, 3, sl)
    idx1 = oracle.select_blocks(q[:, :1], k, 8, 3, sl)
    np.testing.assert_array_equal(idx, idx1)


@pytest.mark.parametrize("lens", [None, [40, 13]])
def test_key_and_value_gradients_by_central_differences(lens):
    L, D = 40, 4
    q, k, v, gate, dout, sl = rand_case(4, B=2 if lens else 1, H=4, Hkv=2, L=L, D=D, lens=lens)
    f = oracle.forward_gqa(q, k, v, gate, 8, 2, 5, sl)
    b = oracle.backward_gqa(q, k, v, gate, 8, 2, 5, f, dout, sl)
    idx = f["idx"]

    def loss(k_, v_):
        return float((oracle.forward_gqa(q, k_, v_, gate, 8, 2, 5, sl, idx=idx)["out"] * dout).sum())

    rng = np.random.default_rng(9)
    h = 1e-5
    for name, arr in (("dk", k), ("dv", v)):
        for _ in range(25):
            pos = tuple(rng.integers(0, s) for s in arr.shape)
            ap, am = arr.copy(), arr.copy()
            ap[pos] += h
            am[pos] -= h
            fd = (loss(ap, v) - loss(am, v)) / (2 * h) if name == "dk" else (loss(k, ap) - loss(k, am)) / (2 * h)
            assert abs(fd - b[name][pos]) < 1e-7 * max(1.0, abs(fd)), (name, pos)
    assert b["dk"].shape == k.shape and b["dq"].shape == q.shape


def test_grouped_selection_through_overlapping_blocks():
    """The paper's full selection (Eq. 8-13: overlapping compression blocks, score remap, scores
    summed over the group's heads): one head per group is the single-head function bit for bit;
    the group scores are the sum of an independent numpy scorer's per-head scores (Eq. 11 as a
    convolution); the chosen set is the stable arg-sort of those sums."""
    from test_oracle_overlap import numpy_scores
    q, k, v, gate, dout, sl = rand_case(6, B=2, H=3, Hkv=3, L=96, D=8, lens=[96, 41])
    idx, sc = oracle.select_blocks_gqa(q, k, 16, 3, sl, return_scores=True, cmp_block=32, cmp_stride=16)
    idx0, sc0, _ = oracle.select_blocks_cmp(q, k, 16, 3, 32, 16, sl, return_scores=True)
    np.testing.assert_array_equal(idx, idx0)
    np.testing.assert_array_equal(sc, sc0)

    q, k, v, gate, dout, sl = rand_case(7, B=2, H=4, Hkv=2, L=96, D=8, lens=[96, 50])
    lp, l, s, topk, scale = 16, 32, 16, 3, 1.0 / math.sqrt(8)
    idx, sc = oracle.select_blocks_gqa(q, k, lp, topk, sl, return_scores=True, cmp_block=l, cmp_stride=s)
    M = 6
    for n in range(2):
        pad0 = 96 - int(sl[n])
        for g in range(2):
            tot = np.zeros((M, M))
            for h in (2 * g, 2 * g + 1):
                tot += numpy_scores(q[n, h], k[n, g], lp, l, s, pad0, scale)[1]
            np.testing.assert_allclose(sc[n, g], tot, atol=1e-12)
            for b in range(M):
                if min((b + 1) * lp, 96) <= max(b * lp, pad0):
                    assert list(idx[n, g, b]) == [-1] * topk
                    continue
                cand = [j for j in range(b) if (j + 1) * lp > pad0]
                order = sorted(cand, key=lambda j: (-tot[b, j], j))[:topk - 1]
                row = sorted(order) + [b]
                assert list(idx[n, g, b][:len(row)]) == row and all(x == -1 for x in idx[n, g, b][len(row):])


def test_heads_must_divide():
    q, k, v, gate, dout, sl = rand_case(5, H=3, Hkv=2)
    with pytest.raises(ValueError):
        oracle.select_blocks_gqa(q, k, 8, 2)
