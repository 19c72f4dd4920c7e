"""Pins of the oracle's selection with overlapping compression blocks (Eq. 8-11, 13).

Independent of the oracle's code: a numpy scorer written from the equations (block means by
slicing, softmax by broadcasting, Eq. 11 as a convolution), the reduction to the plain selection
when the compression blocks coincide with the selection blocks, the worked case of the paper's
default sizes, and invariants of the scores.
"""
import numpy as np
import pytest

from oracle import blossom_oracle as oracle


def rand_qk(seed, B=2, H=2, L=100, D=8):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((B, H, L, D)), rng.standard_normal((B, H, L, D))


def numpy_scores(q, k, lp, l, s, pad0, scale):
    """S_cmp [M, Mc] and S_ltis [M, M] of one (n, h) unit, from Eq. 8-11."""
    L, D = q.shape
    M = -(-L // lp)
    Mc = (L - l) // s + 1 if L >= l else 0
    means = np.zeros((Mc, D))
    live = np.zeros(Mc, dtype=bool)
    for i in range(Mc):
        lo = max(i * s, pad0)
        if lo < i * s + l:
            means[i] = k[lo:i * s + l].mean(axis=0)
            live[i] = True
    S_cmp = np.zeros((M, Mc))
    S_ltis = np.zeros((M, M))
    kern = np.convolve(np.ones(lp // s), np.ones(l // s))       # multiplicities of Eq. 11's double sum
    for b in range(M):
        qlo, qhi = max(b * lp, pad0), min((b + 1) * lp, L)
        if qlo >= qhi:
            continue
        cand = live & (np.arange(Mc) * s + l <= b * lp)
        if cand.any():
            z = scale * q[qlo:qhi] @ means[cand].T
            p = np.exp(z - z.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            S_cmp[b, cand] = p.sum(axis=0)
        # S_ltis[j] = sum_d kern[d] * S_cmp[(lp/s) j - d]: a convolution sampled at (lp/s) j
        if Mc == 0:
            continue
        full = np.convolve(S_cmp[b], kern)                       # full[x] = sum_d kern[d] S_cmp[x - d]
        for j in range(b):
            x = (lp // s) * j
            if x < len(full) and min((j + 1) * lp, L) > max(j * lp, pad0):
                S_ltis[b, j] = full[x]
    return S_cmp, S_ltis


@pytest.mark.parametrize("L,lp,lens", [(100, 16, [100, 37]), (64, 8, None), (50, 16, [50, 9]), (33, 4, [33, 1])])
def test_reduces_to_the_plain_selection(L, lp, lens):
    q, k = rand_qk(1, L=L)
    sl = None if lens is None else np.asarray(lens, dtype=np.int32)
    idx0, sc0 = oracle.select_blocks(q, k, lp, 4, sl, return_scores=True)
    idx1, sc1, _ = oracle.select_blocks_cmp(q, k, lp, 4, lp, lp, sl, return_scores=True)
    np.testing.assert_array_equal(idx0, idx1)
    np.testing.assert_array_equal(sc0, sc1)


@pytest.mark.parametrize("L,lp,l,s,topk,lens", [
    (128, 16, 32, 16, 4, None),          # the paper's default sizes
    (200, 16, 32, 16, 4, [200, 77]),
    (160, 32, 32, 16, 3, [160, 50]),     # two strides per selection block
    (96, 16, 48, 8, 5, None),            # long blocks, small stride
    (90, 8, 8, 4, 3, [90, 31]),
    (20, 16, 32, 16, 4, None),           # shorter than one compression block: no scores at all
])
def test_scores_and_indices_against_the_numpy_scorer(L, lp, l, s, topk, lens):
    q, k = rand_qk(2, L=L)
    B, H, _, D = q.shape
    sl = None if lens is None else np.asarray(lens, dtype=np.int32)
    idx, sc, scc = oracle.select_blocks_cmp(q, k, lp, topk, l, s, sl, return_scores=True)
    M = -(-L // lp)
    for n in range(B):
        pad0 = 0 if sl is None else L - int(sl[n])
        for h in range(H):
            S_cmp, S_ltis = numpy_scores(q[n, h], k[n, h], lp, l, s, pad0, 1.0 / np.sqrt(D))
            np.testing.assert_allclose(scc[n, h], S_cmp, atol=1e-12)
            np.testing.assert_allclose(sc[n, h], S_ltis, atol=1e-12)
            for b in range(M):
                if min((b + 1) * lp, L) <= max(b * lp, pad0):
                    assert np.all(idx[n, h, b] == -1)
                    continue
                livej = [j for j in range(b) if min((j + 1) * lp, L) > max(j * lp, pad0)]
                order = sorted(livej, key=lambda j: (-S_ltis[b, j], j))[:topk - 1]
                want = sorted(order) + [b]
                got = [int(x) for x in idx[n, h, b] if x >= 0]
                # forgive only true near-ties of the two independent evaluations
                if got != want:
                    vals = sorted(S_ltis[b, livej], reverse=True)
                    gap = vals[topk - 2] - vals[topk - 1]
                    assert gap < 1e-9, (n, h, b, got, want)


def test_paper_default_sizes_sum_two_neighbouring_compression_scores():
    """l = 32, s = 16, l' = 16: Eq. 11 has one m and two n terms, S_ltis[j] = S_cmp[j] + S_cmp[j-1]."""
    q, k = rand_qk(3, B=1, H=1, L=256)
    _, sc, scc = oracle.select_blocks_cmp(q, k, 16, 4, 32, 16, return_scores=True)
    M, Mc = sc.shape[-1], scc.shape[-1]
    for b in range(M):
        for j in range(b):
            a = scc[0, 0, b, j] if j < Mc else 0.0
            c = scc[0, 0, b, j - 1] if 1 <= j <= Mc else 0.0
            assert abs(sc[0, 0, b, j] - (a + c)) < 1e-14
    # each valid query spreads a probability mass of one over the candidates
    for b in range(M):
        ncand = sum(1 for i in range(Mc) if i * 16 + 32 <= b * 16)
        assert abs(scc[0, 0, b].sum() - (16.0 if ncand else 0.0)) < 1e-10
        # no compression block that reaches into the query block or beyond is scored
        assert np.all(scc[0, 0, b, ncand:] == 0.0)


def test_without_candidates_the_lowest_blocks_are_taken():
    """Query blocks that start before the first compression block ends have no scores: all past
    selection blocks tie at zero and the tie rule keeps the lowest indices."""
    q, k = rand_qk(4, B=1, H=1, L=128)
    idx = oracle.select_blocks_cmp(q, k, 16, 3, 64, 16)
    assert list(idx[0, 0, 0]) == [0, -1, -1]
    assert list(idx[0, 0, 1]) == [0, 1, -1]
    assert list(idx[0, 0, 2]) == [0, 1, 2]
    assert list(idx[0, 0, 3]) == [0, 1, 3]       # 3 * 16 < 64: still no compression block in the past


def test_bad_sizes_are_rejected():
    q, k = rand_qk(5, L=64)
    for l, s in [(24, 16), (32, 12), (0, 16), (32, 0)]:
        with pytest.raises(ValueError):
            oracle.select_blocks_cmp(q, k, 16, 4, l, s)
