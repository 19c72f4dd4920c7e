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


def _dense(t) -> bool:
    """True if the tensor's elements tile its storage span without gaps or overlap, so that a
    buffer of ``numel`` elements laid out with the same strides holds every element."""
    span = 1 + sum((n - 1) * st for n, st in zip(t.shape, t.stride()) if n > 0)
    return t.numel() > 0 and span == t.numel() and all(st > 0 for st in t.stride())


def _like(t):
    """An uninitialised tensor with exactly t's shape AND strides (``empty_like`` does not keep the
    strides of a non-dense view; the library writes every q-shaped buffer with the strides passed
    in the params)."""
    return torch.empty_strided(t.shape, t.stride(), dtype=t.dtype, device=t.device)


def check_arguments(q, k, v, gate_logits, seq_lens, require_cuda=True, gate_mode=0):
    """Host-side validation before anything is launched: the library receives raw addresses, so a
    host tensor, a tensor on another device, a wrong integer width or a wrong shape would become a
    device memory fault instead of a Python error.  Returns seq_lens as the int32 CUDA tensor the
    library reads (or None).  ``require_cuda=False`` (host-side tests only) skips the test that
    the tensors are CUDA tensors and keeps every other check, the same-device one included."""
    if q.dtype not in _DT or k.dtype != q.dtype or v.dtype != q.dtype:
        raise TypeError("q, k, v must share one dtype, float32 or bfloat16")
    if not ((q.is_cuda or not require_cuda) and q.dim() == 4 and k.dim() == 4 and k.shape == v.shape):
        raise ValueError("q [B, H, L, D] and k, v [B, Hkv, L, D] must be CUDA tensors")
    if k.device != q.device or v.device != q.device:
        raise ValueError("q, k, v must live on one device")
    B, H, L, D = q.shape
    if k.shape[0] != B or k.shape[2] != L or k.shape[3] != D or k.shape[1] < 1 or H % k.shape[1]:
        raise ValueError("k, v must be [B, Hkv, L, D] with Hkv dividing the number of query heads")
    gshape = (H, 2 * D + 1) if gate_mode else (H, 2)
    if not isinstance(gate_logits, torch.Tensor) or tuple(gate_logits.shape) != gshape:
        raise ValueError(f"gate_logits must be a tensor of shape {list(gshape)}")
    if (require_cuda and not gate_logits.is_cuda) or gate_logits.device != q.device:
        raise ValueError("gate_logits must be a CUDA tensor on q's device")
    if not gate_logits.dtype.is_floating_point:
        raise TypeError("gate_logits must be a floating-point tensor")
    if seq_lens is not None:
        if not isinstance(seq_lens, torch.Tensor) or tuple(seq_lens.shape) != (B,):
            raise ValueError("seq_lens must be None or a tensor of shape [B]")
        if seq_lens.dtype not in (torch.int32, torch.int64):
            raise TypeError("seq_lens must be int32 (int64 is converted)")
        if (require_cuda and not seq_lens.is_cuda) or seq_lens.device != q.device:
            raise ValueError("seq_lens must be a CUDA tensor on q's device")
        seq_lens = seq_lens.to(torch.int32).contiguous()
    return seq_lens


class _BlossomAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, gate_logits, seq_lens, block_size, top_k, window, sm_scale,
                stis_mode, stis_block, cmp_block, cmp_stride, per_query=0, phi_logits=None,
                gate_mode=0, causal=1, rope_theta=0.0):
        seq_lens = check_arguments(q, k, v, gate_logits, seq_lens, gate_mode=gate_mode)
        B, H, L, D = q.shape
        Hkv = k.shape[1]
        # The library addresses every q-shaped buffer with q's strides and every k-shaped one with
        # k's: views that are not dense (a slice of a packed projection) are copied first.
        if not (_dense(q) and q.stride(3) == 1):
            q = q.contiguous()
        if not (_dense(k) and k.stride(3) == 1 and k.stride() == v.stride()):
            k, v = k.contiguous(), v.contiguous()
        if Hkv == H and k.stride() != q.stride():
            k, v = _like(q).copy_(k), _like(q).copy_(v)
        params = binding.make_params(B, H, L, D, block_size, top_k, window, _DT[q.dtype],
                                     sm_scale=sm_scale, strides=q.stride()[:3], stis_mode=stis_mode,
                                     stis_block=stis_block, cmp_block=cmp_block, cmp_stride=cmp_stride,
                                     kv_heads=Hkv, kv_strides=k.stride()[:3], select_mode=int(per_query),
                                     phi_logits=phi_logits, gate_mode=int(gate_mode), causal=int(causal),
                                     rope_theta=float(rope_theta))
        nbytes = binding.blossom_workspace_bytes(params)
        if nbytes == 0:
            raise binding.BlossomError(binding.BLOSSOM_ERR_UNSUPPORTED, "blossom_workspace_bytes")
        dev = q.device
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        gate = gate_logits.detach().to(torch.float32).contiguous()
        M = -(-L // block_size)
        idx = torch.empty((B, Hkv, L if per_query else M, top_k), dtype=torch.int32, device=dev)
        out, out_lt, out_st = _like(q), _like(q), _like(q)
        lse = torch.empty((2, B, H, L), dtype=torch.float32, device=dev)
        binding.blossom_attn_fwd(params, q, k, v, gate, seq_lens, idx, 0, out, out_lt, out_st, lse,
                                 workspace)
        ctx.params, ctx.workspace, ctx.seq_lens = params, workspace, seq_lens
        ctx.phi_logits = phi_logits  # the params hold its address: keep it alive until the backward
        ctx.gate_dtype = gate_logits.dtype
        ctx.save_for_backward(q, k, v, gate, idx, out_lt, out_st, lse)
        ctx.mark_non_differentiable(idx)
        return out, idx

    @staticmethod
    def backward(ctx, dout, _didx):
        q, k, v, gate, idx, out_lt, out_st, lse = ctx.saved_tensors
        if dout.stride() != q.stride() or dout.dtype != q.dtype:  # the library wants q's layout
            dout = _like(q).copy_(dout)
        dq, dk, dv = _like(q), _like(k), _like(k)
        dgate = torch.empty(tuple(gate.shape), dtype=torch.float32, device=q.device)
        # the workspace is this call's own and its last user was the training forward above (or an
        # earlier backward, which leaves the lists alone): the backward may reuse that call's tile lists
        params = binding.blossom_params.from_buffer_copy(ctx.params)
        params.reuse_tile_lists = 1
        binding.blossom_attn_bwd(params, q, k, v, gate, ctx.seq_lens, idx, out_lt, out_st, lse,
                                 dout, dq, dk, dv, dgate, ctx.workspace)
        return (dq, dk, dv, dgate.to(ctx.gate_dtype)) + (None,) * 14


def blossom_attention(q, k, v, gate_logits, block_size, top_k, window, seq_lens=None, sm_scale=0.0,
                      return_indices=False, short_term="window", mask_block=1, cmp_block=0,
                      cmp_stride=0, select_per_query=False, phi_logits=None, input_dependent_gate=False, causal=True, rope_theta=0.0):
    """Gated two-branch sparse attention of q [B, H, L, D] and k, v [B, Hkv, L, D] (float32 or
    bfloat16, CUDA; Hkv divides H: with Hkv < H the query heads of a group share key/value head
    and selection, and the returned indices are [B, Hkv, M, top_k]).

    gate_logits: [H, 2] (column 0 long-term, column 1 short-term branch); seq_lens: optional int32
    [B] valid lengths of left-padded sequences; sm_scale 0 means 1/sqrt(D).  Differentiable in
    q, k, v and gate_logits.  Returns the output, and the selected block indices if asked.
    A wait that runs out inside a kernel is reported through ``binding.blossom_device_status`` of
    the call's workspace (it synchronises, so this front end does not poll it).
    short_term: "window" (keys t - window < p <= t) or "power-law" (Eq. 15: the window, blocks of
    mask_block positions at power-of-two block distances, and the last mask_block positions).
    cmp_block / cmp_stride: length and stride of overlapping compression blocks for the selection
    (Eq. 8, 11); 0 = the selection blocks themselves.
    select_per_query: one selection per query position (Eq. 13 as printed; indices [B, Hkv, L,
    top_k]) instead of one per query block.
    input_dependent_gate: Eq. 18's gate with a one-layer F_o: gate_logits is [H, 2 D + 1] = (w_lt,
    w_st, b) per head and alpha = sigmoid(<w_lt, out_lt> + <w_st, out_st> + b) per query row
    (differentiable in those parameters).
    causal: False drops the causal mask (bidirectional encoders): a query block scores every other
    live block, a query sees all valid keys of its selected blocks, Eq. 15 is symmetric.
    rope_theta: > 0 applies rotary position embedding to q and k inside the library (interleaved
    pairs, angle t * rope_theta^(-2i / D)); the gradients returned are those of the unrotated q, k.
    phi_logits: optional float32 CUDA tensor [cmp_block or block_size]: Eq. 9's learnable block
    summary as a softmax pooling over a block's positions (None = the mean).  It only steers the
    selection, which is not differentiated, so it receives no gradient here.
    """
    if phi_logits is not None:
        n = int(cmp_block) or int(block_size)
        if not (isinstance(phi_logits, torch.Tensor) and phi_logits.is_cuda and phi_logits.device == q.device
                and phi_logits.dtype == torch.float32 and tuple(phi_logits.shape) == (n,)):
            raise ValueError(f"phi_logits must be a float32 CUDA tensor of shape [{n}] on q's device")
        phi_logits = phi_logits.detach().contiguous()
    if short_term not in ("window", "power-law"):
        raise ValueError("short_term must be 'window' or 'power-law'")
    out, idx = _BlossomAttention.apply(q, k, v, gate_logits, seq_lens, int(block_size), int(top_k),
                                       int(window), float(sm_scale),
                                       1 if short_term == "power-law" else 0, int(mask_block),
                                       int(cmp_block), int(cmp_stride), int(bool(select_per_query)), phi_logits,
                                       int(bool(input_dependent_gate)), int(bool(causal)), float(rope_theta))
    return (out, idx) if return_indices else out
