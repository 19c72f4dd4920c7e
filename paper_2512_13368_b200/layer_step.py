"""The end-to-end layer case: a 2-layer SASRec-style causal encoder whose self-attention is the
library's gated sparse attention, trained one step on synthetic item sequences.

This module is a measurement harness around the op (PyTorch supplies embeddings, projections,
LayerNorm, the feed-forward block, the loss and autograd; the attention itself runs in the CUDA
library through ``autograd.blossom_attention``).  It exists to time the attention's share of a
full forward + backward step, not to train a recommender.

Shapes of the layer case: hidden 64, 2 heads (head dim 32), feed-forward 256 with GELU, post-LN,
dropout off, item table 50,000 x 64 in bf16, batch 128 x sequence 1024 of item ids drawn from a
Zipf(1.1) law, next-item cross-entropy over 1 positive + 127 uniform negatives per position;
rotary position encoding on q and k; attention hyper-parameters of the mid-length case
(block 32, top-k 8, window 64) since the layer case names none.
"""
from __future__ import annotations

import numpy as np
import torch
import torch.nn as nn
import torch.nn.functional as F

from . import binding
from .autograd import blossom_attention


def zipf_ids(batch, seq_len, n_items, s=1.1, seed=1):
    """[batch, seq_len + 1] int64 item ids in [1, n_items], rank r drawn with weight r^-s."""
    rng = np.random.default_rng(seed)
    w = np.arange(1, n_items + 1, dtype=np.float64) ** (-s)
    return torch.from_numpy(rng.choice(n_items, size=(batch, seq_len + 1), p=w / w.sum()) + 1)


def rope(x):
    """Rotary position encoding of [B, H, L, D] (pairs (2i, 2i+1), base 10000)."""
    B, H, L, D = x.shape
    pos = torch.arange(L, device=x.device, dtype=torch.float32)
    inv = 10000.0 ** (-torch.arange(0, D, 2, device=x.device, dtype=torch.float32) / D)
    ang = pos[:, None] * inv[None, :]
    cos, sin = ang.cos().to(x.dtype), ang.sin().to(x.dtype)
    x0, x1 = x[..., 0::2], x[..., 1::2]
    return torch.stack((x0 * cos - x1 * sin, x0 * sin + x1 * cos), dim=-1).flatten(-2)


class BlossomLayer(nn.Module):
    def __init__(self, hidden, heads, ffn, block, topk, window):
        super().__init__()
        self.heads, self.block, self.topk, self.window = heads, block, topk, window
        self.qkv = nn.Linear(hidden, 3 * hidden)
        self.proj = nn.Linear(hidden, hidden)
        self.gate_logits = nn.Parameter(torch.zeros(heads, 2))
        self.ln1, self.ln2 = nn.LayerNorm(hidden), nn.LayerNorm(hidden)
        self.ff1, self.ff2 = nn.Linear(hidden, ffn), nn.Linear(ffn, hidden)

    def forward(self, x):
        B, L, C = x.shape
        q, k, v = self.qkv(x).view(B, L, 3, self.heads, C // self.heads).permute(2, 0, 3, 1, 4)
        q, k, v = rope(q).contiguous(), rope(k).contiguous(), v.contiguous()
        a = blossom_attention(q, k, v, self.gate_logits, self.block, self.topk, self.window)
        x = self.ln1(x + self.proj(a.transpose(1, 2).reshape(B, L, C)))
        return self.ln2(x + self.ff2(F.gelu(self.ff1(x))))


class BlossomEncoder(nn.Module):
    def __init__(self, n_items=50000, hidden=64, heads=2, ffn=256, layers=2, block=32, topk=8, window=64):
        super().__init__()
        self.emb = nn.Embedding(n_items + 1, hidden, padding_idx=0)
        nn.init.normal_(self.emb.weight, std=0.02)
        self.layers = nn.ModuleList(BlossomLayer(hidden, heads, ffn, block, topk, window) for _ in range(layers))

    def forward(self, ids):
        x = self.emb(ids)
        for layer in self.layers:
            x = layer(x)
        return x

    def loss(self, ids, targets, negatives):
        """Sampled softmax: the positive against `negatives` [B, L, N] uniform item ids."""
        h = self.forward(ids)                                        # [B, L, C]
        cand = torch.cat((targets[..., None], negatives), dim=-1)   # [B, L, 1 + N]
        logits = (h[:, :, None, :] * self.emb(cand)).sum(-1).float()
        return F.cross_entropy(logits.flatten(0, 1), torch.zeros(logits.shape[0] * logits.shape[1],
                                                                 dtype=torch.long, device=ids.device))


def attention_share(batch=128, seq_len=1024, n_items=50000, negatives=127, steps=5, warmup=2,
                    device="cuda:0", seed=1):
    """Times full forward + backward steps of the layer case and the library kernels inside them.

    Returns a dict: ms per step, ms of the library's kernels per step (summed device times from
    the per-launch event profile), their share, and the loss of the last step.
    """
    torch.manual_seed(seed)
    dev = torch.device(device)
    model = BlossomEncoder(n_items=n_items).to(dev).to(torch.bfloat16)
    seq = zipf_ids(batch, seq_len, n_items, seed=seed).to(dev)
    ids, targets = seq[:, :-1], seq[:, 1:]
    g = torch.Generator(device="cpu").manual_seed(seed)
    neg = torch.randint(1, n_items + 1, (batch, seq_len, negatives), generator=g).to(dev)

    def step():
        model.zero_grad(set_to_none=True)
        loss = model.loss(ids, targets, neg)
        loss.backward()
        return loss

    for _ in range(warmup):
        step()
    torch.cuda.synchronize(dev)
    binding.blossom_profile_start(64 * steps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        loss = step()
    e1.record()
    torch.cuda.synchronize(dev)
    launches = binding.blossom_profile_stop(64 * steps)
    total = e0.elapsed_time(e1) / steps
    ours = sum(ms for _, ms in launches) / steps
    return {"ms_per_step": total, "attention_ms_per_step": ours, "attention_share": ours / total,
            "library_launches_per_step": len(launches) / steps, "loss": float(loss.detach())}


if __name__ == "__main__":
    import json
    binding.load()
    print(json.dumps(attention_share()))
