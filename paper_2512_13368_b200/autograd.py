"""``torch.autograd`` front end of the library: ``blossom_attention(q, k, v, gate_logits, ...)``.

Plumbing only: it allocates the outputs and the workspace with PyTorch, calls
``blossom_attn_fwd`` / ``blossom_attn_bwd`` through the C ABI on the current stream and hands the
gradients back to autograd.  Every step of the method runs in the CUDA library; there is no
PyTorch fallback.  The selection is not differentiated (top-k is piecewise constant).
"""
from __future__ import annotations

import torch

from . import binding

_DT = {torch.float32: "fp32", torch.bfloat16: "bf16"}


class _BlossomAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, gate_logits, seq_lens, block_size, top_k, window, sm_scale,
                stis_mode, stis_block, cmp_block, cmp_stride):
        if q.dtype not in _DT or k.dtype != q.dtype or v.dtype != q.dtype:
            raise TypeError("q, k, v must share one dtype, float32 or bfloat16")
        if not (q.is_cuda and q.shape == k.shape == v.shape and q.dim() == 4):
            raise ValueError("q, k, v: CUDA tensors of one shape [B, H, L, D]")
        if not (q.stride() == k.stride() == v.stride() and q.stride(3) == 1):
            q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        B, H, L, D = q.shape
        params = binding.make_params(B, H, L, D, block_size, top_k, window, _DT[q.dtype],
                                     sm_scale=sm_scale, strides=q.stride()[:3], stis_mode=stis_mode,
                                     stis_block=stis_block, cmp_block=cmp_block, cmp_stride=cmp_stride)
        nbytes = binding.blossom_workspace_bytes(params)
        if nbytes == 0:
            raise binding.BlossomError(binding.BLOSSOM_ERR_UNSUPPORTED, "blossom_workspace_bytes")
        dev = q.device
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        gate = gate_logits.detach().to(torch.float32).contiguous()
        M = -(-L // block_size)
        idx = torch.empty((B, H, M, top_k), dtype=torch.int32, device=dev)
        out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=dev)
        out_lt, out_st = torch.empty_like(out), torch.empty_like(out)
        lse = torch.empty((2, B, H, L), dtype=torch.float32, device=dev)
        binding.blossom_attn_fwd(params, q, k, v, gate, seq_lens, idx, 0, out, out_lt, out_st, lse,
                                 workspace)
        ctx.params, ctx.workspace, ctx.seq_lens = params, workspace, seq_lens
        ctx.gate_dtype = gate_logits.dtype
        ctx.save_for_backward(q, k, v, gate, idx, out_lt, out_st, lse)
        ctx.mark_non_differentiable(idx)
        return out, idx

    @staticmethod
    def backward(ctx, dout, _didx):
        q, k, v, gate, idx, out_lt, out_st, lse = ctx.saved_tensors
        if dout.stride() != q.stride() or dout.dtype != q.dtype:  # the library wants q's layout
            tmp = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=q.device)
            tmp.copy_(dout)
            dout = tmp
        dq, dk, dv = torch.empty_like(out_lt), torch.empty_like(out_lt), torch.empty_like(out_lt)
        dgate = torch.empty((q.shape[1], 2), dtype=torch.float32, device=q.device)
        binding.blossom_attn_bwd(ctx.params, q, k, v, gate, ctx.seq_lens, idx, out_lt, out_st, lse,
                                 dout, dq, dk, dv, dgate, ctx.workspace)
        return dq, dk, dv, dgate.to(ctx.gate_dtype), None, None, None, None, None, None, None, None, None


def blossom_attention(q, k, v, gate_logits, block_size, top_k, window, seq_lens=None, sm_scale=0.0,
                      return_indices=False, short_term="window", mask_block=1, cmp_block=0,
                      cmp_stride=0):
    """Gated two-branch sparse attention of [B, H, L, D] tensors (float32 or bfloat16, CUDA).

    gate_logits: [H, 2] (column 0 long-term, column 1 short-term branch); seq_lens: optional int32
    [B] valid lengths of left-padded sequences; sm_scale 0 means 1/sqrt(D).  Differentiable in
    q, k, v and gate_logits.  Returns the output, and the selected block indices if asked.
    short_term: "window" (keys t - window < p <= t) or "power-law" (Eq. 15: the window, blocks of
    mask_block positions at power-of-two block distances, and the last mask_block positions).
    cmp_block / cmp_stride: length and stride of overlapping compression blocks for the selection
    (Eq. 8, 11); 0 = the selection blocks themselves.
    """
    if short_term not in ("window", "power-law"):
        raise ValueError("short_term must be 'window' or 'power-law'")
    out, idx = _BlossomAttention.apply(q, k, v, gate_logits, seq_lens, int(block_size), int(top_k),
                                       int(window), float(sm_scale),
                                       1 if short_term == "power-law" else 0, int(mask_block),
                                       int(cmp_block), int(cmp_stride))
    return (out, idx) if return_indices else out
