"""Seeded synthetic inputs for the BlossomRec sparse-attention path.

This module only draws random numbers and rounds them to the storage type; it
holds none of the method's arithmetic, so that both the CUDA library's tests and
the independent CPU checker can be fed the identical bytes.

Recommendation-shaped batches: short head dims (32 / 64), few heads, many
sequences, left padding with widely varying lengths.  They stand in for the
public interaction logs the paper trains on (which are not redistributed here).

Draw order for every workload (numpy ``default_rng(seed)``, float32):
q, k, v, gate logits, upstream gradient, then the workload's extras
(sequence lengths or per-row scales).  Values are rounded once (nearest-even) to
the storage dtype and handed out as float32 arrays holding exactly those values.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


def round_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> float32 holding the same values."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def quantize(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float32 array to ``dtype`` ('fp32' or 'bf16'); result is float32."""
    if dtype == "fp32":
        return np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "bf16":
        return bf16_bits_to_f32(round_to_bf16_bits(x)).reshape(x.shape)
    raise ValueError(dtype)


@dataclass
class Workload:
    name: str
    dtype: str            # 'fp32' | 'bf16' : storage type of q, k, v, out, dout, dq, dk, dv
    B: int
    H: int
    L: int
    D: int
    block: int
    topk: int
    window: int
    seed: int
    q: np.ndarray = field(repr=False)
    k: np.ndarray = field(repr=False)
    v: np.ndarray = field(repr=False)
    gate: np.ndarray = field(repr=False)      # [H, 2] float32
    dout: np.ndarray = field(repr=False)
    seq_lens: np.ndarray | None = field(default=None, repr=False)  # [B] int32 or None
    stis_mode: int = 0    # short-term branch: 0 = causal window, 1 = power-law mask (Eq. 15)
    stis_block: int = 1   # mask block of the power-law mask
    cmp_block: int = 0    # compression block length l of the selection (0 = block)
    cmp_stride: int = 0   # and its stride s (0 = block)
    kv_heads: int = 0     # key/value heads (0 = H): k, v are [B, kv_heads, L, D]
    per_query: int = 0    # 1: one selection per query position (Eq. 13 as printed) instead of per query block
    phi_logits: np.ndarray | None = field(default=None, repr=False)  # learnable block summary (Eq. 9) or None = mean
    gate_mode: int = 0    # 1: Eq. 18's input-dependent gate, gate is [H, 2 D + 1] = (w_lt, w_st, b)
    causal: int = 1       # 0: no causal mask (bidirectional encoder)
    rope_theta: float = 0.0  # > 0: q and k are rotated by position inside the library

    @property
    def n_blocks(self) -> int:
        return -(-self.L // self.block)

    @property
    def tokens(self) -> int:
        return self.B * self.L

    def unit(self, n: int, h: int) -> "Workload":
        """The single (batch n, key/value head h) problem as a B=1 workload: one head, or with
        grouped heads the query heads that share key/value head h."""
        sl = None if self.seq_lens is None else self.seq_lens[n:n + 1].copy()
        G = self.H // (self.kv_heads or self.H)
        hq = slice(h * G, (h + 1) * G)
        return Workload(self.name + f"[{n},{h}]", self.dtype, 1, G, self.L, self.D, self.block,
                        self.topk, self.window, self.seed,
                        self.q[n:n + 1, hq].copy(), self.k[n:n + 1, h:h + 1].copy(),
                        self.v[n:n + 1, h:h + 1].copy(), self.gate[hq].copy(),
                        self.dout[n:n + 1, hq].copy(), sl, self.stis_mode, self.stis_block,
                        self.cmp_block, self.cmp_stride, 1 if G > 1 else 0, self.per_query, self.phi_logits, self.gate_mode, self.causal, self.rope_theta)


def make(name, dtype, B, H, L, D, block, topk, window, seed, std=1.0, lengths=None,
         row_scales=False, stis_mode=0, stis_block=1, kv_heads=0) -> Workload:
    """Generic generator; see the module docstring for the draw order.

    lengths: None or (lo, hi) inclusive -> left-padded sequences, pad rows keep their
    random contents (they must not influence any result).
    row_scales: multiply every row of q, k, v by its own U(0.5, 2) factor.
    """
    rng = np.random.default_rng(seed)
    shape = (B, H, L, D)
    kv_shape = (B, kv_heads or H, L, D)
    q = rng.standard_normal(shape, dtype=np.float32) * np.float32(std)
    k = rng.standard_normal(kv_shape, dtype=np.float32) * np.float32(std)
    v = rng.standard_normal(kv_shape, dtype=np.float32) * np.float32(std)
    gate = rng.standard_normal((H, 2), dtype=np.float32)
    dout = rng.standard_normal(shape, dtype=np.float32)
    seq_lens = None
    if lengths is not None:
        lo, hi = lengths
        seq_lens = rng.integers(lo, hi + 1, size=(B,), dtype=np.int64).astype(np.int32)
    if row_scales:
        for t in (q, k, v):
            t *= rng.uniform(0.5, 2.0, size=t.shape[:3] + (1,)).astype(np.float32)
    return Workload(name, dtype, B, H, L, D, block, topk, window, seed,
                    quantize(q, dtype), quantize(k, dtype), quantize(v, dtype),
                    gate, quantize(dout, dtype), seq_lens, stis_mode, stis_block, 0, 0, kv_heads)


# The five benchmark configurations.
def config1() -> Workload:
    """tiny fp32 correctness case: B4 H2 L64 D32, block 8, top-k 2, window 16, seed 0."""
    return make("cfg1-tiny-fp32", "fp32", 4, 2, 64, 32, 8, 2, 16, seed=0)


def config2(B: int = 256, kv_heads: int = 0) -> Workload:
    """short-sequence batch: bf16, L200 D32, block 16, top-k 4, window 32, lengths U{5..200}."""
    return make("cfg2-short-padded", "bf16", B, 2, 200, 32, 16, 4, 32, seed=2, std=0.5,
                lengths=(5, 200), kv_heads=kv_heads)


def config3(B: int = 128, kv_heads: int = 0) -> Workload:
    """mid-length: bf16, H4 L1024 D64, block 32, top-k 8, window 64, per-row norm scales."""
    return make("cfg3-mid", "bf16", B, 4, 1024, 64, 32, 8, 64, seed=3, row_scales=True, kv_heads=kv_heads)


def config4(B: int = 16, kv_heads: int = 0) -> Workload:
    """long-history headline: bf16, H8 L4096 D64, block 64, top-k 16, window 256."""
    return make("cfg4-long", "bf16", B, 8, 4096, 64, 64, 16, 256, seed=4, kv_heads=kv_heads)


def config5_attention(B: int = 128, kv_heads: int = 0) -> Workload:
    """attention-shaped slice of the end-to-end layer case: bf16, H2 L1024 D32, block 32,
    top-k 8, window 64 (the layer case gives no attention hyper-parameters; the mid-length
    case's are reused)."""
    return make("cfg5-layer-attn", "bf16", B, 2, 1024, 32, 32, 8, 64, seed=1, kv_heads=kv_heads)


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5_attention}
