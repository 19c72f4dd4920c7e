"""Pins of the oracle's power-law short-term mask (Eq. 15 with all three cases, causal side).

None of these re-uses the oracle's own code: the mask is rebuilt from Eq. 15 with numpy
broadcasting, row populations are compared with closed forms, limiting cases reduce to dense
causal attention, and the backward is checked by central differences.
"""
import math

import numpy as np
import pytest

from oracle import blossom_oracle as oracle


def rand_case(seed, B=2, H=2, L=40, D=8, lens=None):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, H, L, D))
    k = rng.standard_normal((B, H, L, D))
    v = rng.standard_normal((B, H, L, D))
    gate = rng.standard_normal((H, 2))
    dout = rng.standard_normal((B, H, L, D))
    sl = None if lens is None else np.asarray(lens, dtype=np.int32)
    return q, k, v, gate, dout, sl


def eq15_mask(L, w, blk):
    """M_STIS of Eq. 15 as a dense [L, L] boolean matrix (no causality, no padding)."""
    i = np.arange(L)[:, None]
    j = np.arange(L)[None, :]
    near = np.abs(i - j) < w
    bd = np.abs(i // blk - j // blk)
    pow2 = (bd >= 1) & ((bd & (bd - 1)) == 0)
    last = np.broadcast_to(j >= L - blk, (L, L))
    return near | pow2 | last


def masked_attention(q, k, v, mask, scale):
    s = np.einsum("bhtd,bhpd->bhtp", q, k) * scale
    s = np.where(mask, s, -np.inf)
    mx = np.max(s, axis=-1, keepdims=True)
    mx = np.where(np.isfinite(mx), mx, 0.0)
    e = np.exp(s - mx)
    den = e.sum(-1, keepdims=True)
    any_ = mask.any(-1, keepdims=True)
    p = np.where(any_, e / np.where(any_, den, 1.0), 0.0)
    lse = np.where(any_[..., 0], mx[..., 0] + np.log(np.where(any_, den, 1.0))[..., 0], 0.0)
    return np.einsum("bhtp,bhpd->bhtd", p, v), lse


@pytest.mark.parametrize("L,w,blk,lens", [
    (40, 3, 1, None),
    (64, 8, 1, [64, 21]),
    (50, 4, 2, [50, 7]),
    (70, 6, 3, None),        # window not a multiple of the mask block, ragged last block
    (33, 1, 1, [33, 2]),
    (48, 8, 4, [48, 30]),
])
def test_short_term_branch_equals_dense_mask_evaluation(L, w, blk, lens):
    q, k, v, gate, dout, sl = rand_case(3, L=L, lens=lens)
    B, H, _, D = q.shape
    f = oracle.forward(q, k, v, gate, 8, 2, w, sl, stis_mode=1, stis_block=blk)
    t = np.arange(L)[:, None]
    p = np.arange(L)[None, :]
    m = np.zeros((B, H, L, L), dtype=bool)
    for n in range(B):
        pad0 = 0 if sl is None else L - int(sl[n])
        m[n, :] = eq15_mask(L, w, blk) & (p <= t) & (t >= pad0) & (p >= pad0)
    o, lse = masked_attention(q, k, v, m, 1.0 / math.sqrt(D))
    np.testing.assert_allclose(f["out_st"], o, atol=1e-12)
    np.testing.assert_allclose(f["lse"][1], lse, atol=1e-12)
    # the long-term branch does not depend on the short-term mode
    g = oracle.forward(q, k, v, gate, 8, 2, w, sl)
    np.testing.assert_array_equal(f["out_lt"], g["out_lt"])
    np.testing.assert_array_equal(f["idx"], g["idx"])


def test_row_populations_closed_form():
    """With q = 0 every visible key has the same weight, so exp(lse) counts a row's keys.

    Mask block 1, window w: row t sees min(t + 1, w) window keys plus one key per power of two
    2^r with w <= 2^r <= t (smaller powers lie inside the window).  For the four lengths of the
    paper's Table 5 and its window of 8 the last row therefore sees w + log2(L) - log2(w) keys:
    the table's log2(L) links minus the log2(w) of them the window already covers.
    """
    D = 4
    for L, w in [(256, 8), (512, 8), (1024, 8), (2048, 8), (128, 1), (100, 5)]:
        rng = np.random.default_rng(L)
        q = np.zeros((1, 1, L, D))
        k = rng.standard_normal((1, 1, L, D))
        v = rng.standard_normal((1, 1, L, D))
        f = oracle.forward(q, k, v, np.zeros((1, 2)), 16, 2, w, stis_mode=1, stis_block=1)
        n_seen = np.exp(f["lse"][1, 0, 0])
        t = np.arange(L)
        expect = np.minimum(t + 1, w).astype(float)
        r = 0
        while (1 << r) < L:
            if (1 << r) >= w:
                expect += (t >= (1 << r))
            r += 1
        np.testing.assert_allclose(n_seen, expect, rtol=1e-12)
        if L in (256, 512, 1024, 2048):
            assert round(n_seen[-1]) == w + int(math.log2(L)) - int(math.log2(w))


def test_limits_reduce_to_dense_causal_and_to_the_window():
    q, k, v, gate, dout, sl = rand_case(5, L=48, lens=[48, 19])
    L = 48
    dense = oracle.forward(q, k, v, gate, 8, 2, L, sl)                       # window = L: dense causal
    a = oracle.forward(q, k, v, gate, 8, 2, L, sl, stis_mode=1, stis_block=1)
    np.testing.assert_allclose(a["out_st"], dense["out_st"], atol=1e-13)
    # mask block >= L: every position lies in "the last blk positions" -> dense causal again
    b = oracle.forward(q, k, v, gate, 8, 2, 1, sl, stis_mode=1, stis_block=L)
    np.testing.assert_allclose(b["out_st"], dense["out_st"], atol=1e-13)
    # blk = 16, L = 48: the only block distances are 1 and 2, both powers of two, so a row sees
    # every earlier block in full; inside its own block (distance 0) it sees its window of 4,
    # except in the last block, all of whose positions up to the row itself are visible
    c = oracle.forward(np.zeros_like(q), k, v, gate, 8, 2, 4, None, stis_mode=1, stis_block=16)
    n_seen = np.exp(c["lse"][1, 0, 0])
    t = np.arange(L)
    own = np.where(t >= 32, t % 16 + 1, np.minimum(t % 16 + 1, 4))
    np.testing.assert_allclose(n_seen, (t // 16) * 16 + own, rtol=1e-12)


@pytest.mark.parametrize("blk,w,lens", [(1, 3, None), (2, 4, [23, 30])])
def test_backward_matches_central_differences(blk, w, lens):
    L, D = 30, 4
    q, k, v, gate, dout, sl = rand_case(7, B=2 if lens else 1, H=1, L=L, D=D, lens=lens)
    f = oracle.forward_backward(q, k, v, gate, dout, 8, 2, w, sl, stis_mode=1, stis_block=blk)
    idx = f["idx"]

    def loss(q_, k_, v_, g_):
        return float((oracle.forward(q_, k_, v_, g_, 8, 2, w, sl, idx=idx, stis_mode=1,
                                     stis_block=blk)["out"] * dout).sum())

    rng = np.random.default_rng(11)
    h = 1e-5
    for name, arr in (("dq", q), ("dk", k), ("dv", v)):
        for _ in range(25):
            pos = tuple(rng.integers(0, s) for s in arr.shape)
            ap, am = arr.copy(), arr.copy()
            ap[pos] += h
            am[pos] -= h
            args_p = {"dq": (ap, k, v, gate), "dk": (q, ap, v, gate), "dv": (q, k, ap, gate)}[name]
            args_m = {"dq": (am, k, v, gate), "dk": (q, am, v, gate), "dv": (q, k, am, gate)}[name]
            fd = (loss(*args_p) - loss(*args_m)) / (2 * h)
            assert abs(fd - f[name][pos]) < 1e-7 * max(1.0, abs(fd)), (name, pos)
    for pos in [(0, 0), (0, 1)]:
        gp, gm = gate.copy(), gate.copy()
        gp[pos] += h
        gm[pos] -= h
        fd = (loss(q, k, v, gp) - loss(q, k, v, gm)) / (2 * h)
        assert abs(fd - f["dgate"][pos]) < 1e-7 * max(1.0, abs(fd))


def test_bad_mode_arguments_are_rejected():
    q, k, v, gate, dout, sl = rand_case(1, L=16)
    with pytest.raises(ValueError):
        oracle.forward(q, k, v, gate, 8, 2, 4, stis_mode=2)
    with pytest.raises(ValueError):
        oracle.forward(q, k, v, gate, 8, 2, 4, stis_mode=1, stis_block=0)
