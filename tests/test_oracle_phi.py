"""Pins of the oracle's learnable block summary (Eq. 9 read as a softmax pooling over the positions
of a block): zero logits are the mean bit for bit, a numpy evaluation written from the formula,
the one-hot limit, invariance to a constant added to the logits, padding."""
import math

import numpy as np
import pytest

from oracle import blossom_oracle as oracle


def rand_qk(seed, B=2, H=2, L=96, D=8):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((B, H, L, D)), rng.standard_normal((B, H, L, D))


def test_zero_logits_are_the_mean_bit_for_bit():
    q, k = rand_qk(1)
    sl = np.asarray([96, 41], dtype=np.int32)
    for fn, args, n in ((oracle.select_blocks, (16, 4), 16), (oracle.select_blocks_per_query, (16, 4), 16)):
        a = fn(q, k, *args, sl, return_scores=True)
        b = fn(q, k, *args, sl, return_scores=True, phi_logits=np.zeros(n))
        np.testing.assert_array_equal(a[0], b[0])
        np.testing.assert_array_equal(a[1], b[1])
    a = oracle.select_blocks_cmp(q, k, 16, 4, 32, 16, sl, return_scores=True)
    b = oracle.select_blocks_cmp(q, k, 16, 4, 32, 16, sl, return_scores=True, phi_logits=np.zeros(32))
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)


@pytest.mark.parametrize("lens", [None, [80, 27]])
def test_scores_from_a_numpy_softmax_pooling(lens):
    L, Bk, D = 80, 16, 8
    q, k = rand_qk(2, L=L, D=D)
    rng = np.random.default_rng(5)
    phi = rng.standard_normal(Bk)
    sl = None if lens is None else np.asarray(lens, dtype=np.int32)
    idx, sc = oracle.select_blocks(q, k, Bk, 3, sl, return_scores=True, phi_logits=phi)
    M = L // Bk
    for n in range(2):
        pad0 = 0 if sl is None else L - int(sl[n])
        for h in range(2):
            means, live = np.zeros((M, D)), np.zeros(M, dtype=bool)
            for j in range(M):
                lo, hi = max(j * Bk, pad0), (j + 1) * Bk
                if lo < hi:
                    w = np.exp(phi[lo - j * Bk:hi - j * Bk])
                    means[j] = (w[:, None] * k[n, h, lo:hi]).sum(axis=0) / w.sum()
                    live[j] = True
            for b in range(1, M):
                qlo = max(b * Bk, pad0)
                cand = [j for j in range(b) if live[j]]
                if qlo >= (b + 1) * Bk or not cand:
                    continue
                z = (q[n, h, qlo:(b + 1) * Bk] @ means[cand].T) / math.sqrt(D)
                p = np.exp(z - z.max(axis=1, keepdims=True))
                p /= p.sum(axis=1, keepdims=True)
                np.testing.assert_allclose(sc[n, h, b, cand], p.sum(axis=0), atol=1e-12)
                keep = sorted(sorted(cand, key=lambda j: (-p.sum(axis=0)[cand.index(j)], j))[:2]) + [b]
                assert list(idx[n, h, b][:len(keep)]) == keep


def test_one_hot_limit_and_shift_invariance():
    q, k = rand_qk(3, B=1, H=1, L=64)
    phi = np.zeros(8)
    phi[5] = 60.0                                   # the summary of a block is its sixth key
    _, sc = oracle.select_blocks(q, k, 8, 3, return_scores=True, phi_logits=phi)
    k2 = np.repeat(k[:, :, 5::8], 8, axis=2)        # every key of a block replaced by that key
    _, sc2 = oracle.select_blocks(q, k2, 8, 3, return_scores=True)
    np.testing.assert_allclose(sc, sc2, atol=1e-12)
    rng = np.random.default_rng(7)
    a = rng.standard_normal(8)
    i1, s1 = oracle.select_blocks(q, k, 8, 3, return_scores=True, phi_logits=a)
    i2, s2 = oracle.select_blocks(q, k, 8, 3, return_scores=True, phi_logits=a + 3.25)
    np.testing.assert_array_equal(i1, i2)
    np.testing.assert_allclose(s1, s2, atol=1e-12)
