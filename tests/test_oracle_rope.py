"""Pins of the oracle's rotary position embedding: the complex-multiplication form, norms, the
relative-position property that makes it a position encoding, the transpose, exact rounding to
bfloat16, and the gradient of the whole path through the rotation by central differences."""
import numpy as np

from oracle import blossom_oracle as oracle


def test_is_multiplication_by_unit_complex_numbers():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 3, 17, 8))
    theta = 10000.0
    z = x[..., 0::2] + 1j * x[..., 1::2]
    ang = np.arange(17)[:, None] * theta ** (-2.0 * np.arange(4) / 8)[None, :]
    zr = z * np.exp(1j * ang)
    y = oracle.rope(x, theta)
    np.testing.assert_allclose(y[..., 0::2], zr.real, atol=1e-13)
    np.testing.assert_allclose(y[..., 1::2], zr.imag, atol=1e-13)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), atol=1e-12)
    np.testing.assert_allclose(oracle.rope(y, theta, transpose=True), x, atol=1e-12)
    np.testing.assert_array_equal(y[..., 0, :], x[..., 0, :])            # position 0 is not rotated


def test_logits_depend_on_the_distance_only():
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal(8), rng.standard_normal(8)
    L = 40
    Q = oracle.rope(np.tile(q, (L, 1)), 500.0)
    K = oracle.rope(np.tile(k, (L, 1)), 500.0)
    S = Q @ K.T
    for d in (0, 1, 7):
        diag = np.array([S[t, t - d] for t in range(d, L)])
        np.testing.assert_allclose(diag, diag[0], atol=1e-12)


def test_rounding_to_bfloat16_is_to_nearest_even():
    from paper_2512_13368_b200 import workloads
    rng = np.random.default_rng(3)
    x = rng.standard_normal(20000) * 10.0 ** rng.integers(-3, 4, 20000)
    r = oracle._round_to_bf16(x)
    assert np.array_equal(r, workloads.quantize(r.astype(np.float32), "bf16").astype(np.float64))   # representable
    # no other bfloat16 value is closer: the neighbours one unit in the last place away
    u = r.astype(np.float32).view(np.uint32)
    nb1 = (u + np.uint32(0x10000)).view(np.float32).astype(np.float64)
    nb0 = (u - np.uint32(0x10000)).view(np.float32).astype(np.float64)
    assert np.all(np.abs(x - r) <= np.abs(x - nb1)) and np.all(np.abs(x - r) <= np.abs(x - nb0))
    assert oracle._round_to_bf16(np.array([1.00390625]))[0] == 1.0            # tie: 1 + 2^-8 -> even
    assert oracle._round_to_bf16(np.array([1.01171875]))[0] == 1.015625       # tie: 1 + 3 * 2^-8 -> even


def test_gradient_through_the_rotation_by_central_differences():
    rng = np.random.default_rng(4)
    B, H, L, D = 1, 2, 24, 4
    q, k, v, dout = (rng.standard_normal((B, H, L, D)) for _ in range(4))
    gate = rng.standard_normal((H, 2))
    theta = 100.0
    f = oracle.forward(oracle.rope(q, theta), oracle.rope(k, theta), v, gate, 8, 2, 5)
    g = oracle.backward(oracle.rope(q, theta), oracle.rope(k, theta), v, gate, 8, 2, 5, f, dout)
    dq = oracle.rope(g["dq"], theta, transpose=True)
    dk = oracle.rope(g["dk"], theta, transpose=True)

    def loss(q_, k_):
        return float((oracle.forward(oracle.rope(q_, theta), oracle.rope(k_, theta), v, gate, 8, 2, 5,
                                     idx=f["idx"])["out"] * dout).sum())

    h = 1e-5
    for arr, grad, which in ((q, dq, 0), (k, dk, 1)):
        for _ in range(20):
            pos = tuple(int(rng.integers(0, n)) for n in arr.shape)
            ap, am = arr.copy(), arr.copy()
            ap[pos] += h
            am[pos] -= h
            fd = (loss(ap, k) - loss(am, k)) / (2 * h) if which == 0 else (loss(q, ap) - loss(q, am)) / (2 * h)
            assert abs(fd - grad[pos]) < 2e-7 * max(1.0, abs(fd)), (which, pos)
