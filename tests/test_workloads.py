"""Seeded input generators: determinism, exact storage-type rounding, recipe shapes."""
import numpy as np
import torch

from paper_2512_13368_b200 import workloads as W


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(20000) * 10 ** rng.uniform(-6, 6, 20000)).astype(np.float32)
    x[:4] = [0.0, -0.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8]   # exact ties go to even
    ours = W.quantize(x, "bf16")
    ref = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    assert np.array_equal(ours.view(np.uint32), ref.view(np.uint32))
    assert np.array_equal(W.quantize(ours, "bf16"), ours)


def test_configs_are_deterministic_and_shaped():
    a, b = W.config1(), W.config1()
    for k in ("q", "k", "v", "gate", "dout"):
        assert np.array_equal(getattr(a, k), getattr(b, k))
    assert (a.B, a.H, a.L, a.D, a.block, a.topk, a.window, a.dtype) == (4, 2, 64, 32, 8, 2, 16, "fp32")
    c2 = W.config2(B=64)
    assert c2.seq_lens.min() >= 5 and c2.seq_lens.max() <= 200 and c2.n_blocks == 13
    assert abs(float(c2.q.std()) - 0.5) < 0.01
    c3 = W.config3(B=1)
    norms = np.linalg.norm(c3.q, axis=-1) / 8.0
    assert norms.min() < 0.6 and norms.max() > 1.9          # per-row scales U(0.5, 2)
    u = c3.unit(0, 2)
    assert u.q.shape == (1, 1, 1024, 64) and np.array_equal(u.gate[0], c3.gate[2])
