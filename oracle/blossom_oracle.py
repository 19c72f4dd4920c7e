"""ctypes front end of the fp64 C oracle (``blossom_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Every function widens its inputs to float64 and calls
the plain-C restatement of the paper's equations; nothing here is shared with
the CUDA library.

Shapes: q, k, v, dout ``[B, H, L, D]``; gate ``[H, 2]`` (column 0 = long-term
branch logit, column 1 = short-term branch logit); seq_lens ``[B]`` valid
lengths of left-padded sequences or ``None``; idx ``[B, H, M, topk]`` int32,
ascending, -1 padded, ``M = ceil(L / block)``.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "blossom_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libblossom_oracle.so")
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2 -fopenmp) if it is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    os.makedirs(os.path.dirname(_LIB), exist_ok=True)
    tmp = _LIB + ".tmp.%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-std=c99", "-fPIC", "-shared",
                           "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i = ctypes.c_int
        d = ctypes.c_double
        lib.blossom_oracle_threads.restype = i
        lib.blossom_oracle_select.restype = i
        lib.blossom_oracle_select.argtypes = [i, i, i, i, i, i, i, d, _dp, _dp, _ip, _dp, _ip, _dp]
        lib.blossom_oracle_select_cmp.restype = i
        lib.blossom_oracle_select_cmp.argtypes = [i, i, i, i, i, i, i, i, d, _dp, _dp, _ip, _dp, _ip, _dp, _dp]
        lib.blossom_oracle_forward.restype = i
        lib.blossom_oracle_select_pq.restype = i
        lib.blossom_oracle_select_pq.argtypes = [i, i, i, i, i, i, d, _dp, _dp, _ip, _dp, _ip, _dp]
        lib.blossom_oracle_select_pq_cmp.restype = i
        lib.blossom_oracle_select_pq_cmp.argtypes = [i, i, i, i, i, i, i, i, d, _dp, _dp, _ip, _dp, _ip, _dp]
        lib.blossom_oracle_forward.argtypes = [i, i, i, i, i, i, i, i, i, i, i, i, d, _dp, _dp, _dp, _dp, _ip,
                                               _ip, _dp, _dp, _dp, _dp]
        lib.blossom_oracle_backward.restype = i
        lib.blossom_oracle_backward.argtypes = [i, i, i, i, i, i, i, i, i, i, i, i, d, _dp, _dp, _dp, _dp, _ip,
                                                _ip, _dp, _dp, _dp, _dp, _dp, _dp, _dp, _dp]
        _lib = lib
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle uses (parallel over (batch, head) only)."""
    return int(_load().blossom_oracle_threads())


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a, ty):
    return a.ctypes.data_as(ty) if a is not None else None


def _lens(seq_lens, B):
    if seq_lens is None:
        return None
    s = np.ascontiguousarray(np.asarray(seq_lens, dtype=np.int32))
    assert s.shape == (B,)
    return s


def _phi(phi_logits, length):
    """The logits of the learnable block summary (softmax pooling over a block's positions), or
    None for the mean."""
    if phi_logits is None:
        return None
    p = np.ascontiguousarray(np.asarray(phi_logits, dtype=np.float64))
    assert p.shape == (length,)
    return p


def _scale(sm_scale, D):
    return float(sm_scale) if sm_scale else 1.0 / math.sqrt(D)


def select_blocks(q, k, block, topk, seq_lens=None, sm_scale=None, return_scores=False, phi_logits=None,
                  causal=True):
    """Eq. 8-10, 12, 13: block summaries, block scores and the top-k block set.

    ``phi_logits`` ``[block]``: Eq. 9's learnable summary as a softmax pooling over the positions of
    a block (weights exp(phi_logits[i]) over the valid keys); None = the mean.
    ``causal=False`` (a bidirectional encoder): a query block scores every live block but itself."""
    q, k = _f64(q), _f64(k)
    B, H, L, D = q.shape
    M = -(-L // block)
    idx = np.empty((B, H, M, topk), dtype=np.int32)
    scores = np.zeros((B, H, M, M), dtype=np.float64) if return_scores else None
    sl = _lens(seq_lens, B)
    ph = _phi(phi_logits, block)
    rc = _load().blossom_oracle_select(B, H, L, D, block, topk, int(bool(causal)), _scale(sm_scale, D),
                                       _ptr(q, _dp), _ptr(k, _dp), _ptr(sl, _ip), _ptr(ph, _dp),
                                       _ptr(idx, _ip), _ptr(scores, _dp))
    if rc:
        raise ValueError("blossom_oracle_select: bad arguments")
    return (idx, scores) if return_scores else idx


def select_blocks_per_query(q, k, block, topk, seq_lens=None, sm_scale=None, return_scores=False,
                            phi_logits=None, cmp_block=0, cmp_stride=0):
    """Eq. 8-10, 13 as printed: one selection per query position.  k may have fewer heads than q
    (grouped heads: the probabilities of a group's heads are summed, Eq. 12, and the group's
    queries at one position share the selection).  With ``cmp_block`` / ``cmp_stride`` the position
    scores overlapping compression blocks and Eq. 11 maps its probabilities onto the selection
    blocks (the paper's selection in full).  Returns idx ``[B,Hkv,L,topk]`` (ascending, -1
    padded, the position's own block included) and, if asked, the (mapped) probabilities
    ``[B,Hkv,L,M]``."""
    q, k = _f64(q), _f64(k)
    B, H, L, D = q.shape
    Hkv = k.shape[1]
    G = _group(H, Hkv)
    M = -(-L // block)
    idx = np.empty((B, H, L, topk), dtype=np.int32)
    probs = np.zeros((B, H, L, M), dtype=np.float64) if (return_scores or G > 1) else None
    sl = _lens(seq_lens, B)
    kk = np.ascontiguousarray(np.repeat(k, G, axis=1))
    if cmp_block or cmp_stride:
        l, s = int(cmp_block or block), int(cmp_stride or block)
        ph = _phi(phi_logits, l)
        rc = _load().blossom_oracle_select_pq_cmp(B, H, L, D, block, topk, l, s, _scale(sm_scale, D),
                                                  _ptr(q, _dp), _ptr(kk, _dp), _ptr(sl, _ip), _ptr(ph, _dp),
                                                  _ptr(idx, _ip), _ptr(probs, _dp))
    else:
        ph = _phi(phi_logits, block)
        rc = _load().blossom_oracle_select_pq(B, H, L, D, block, topk, _scale(sm_scale, D), _ptr(q, _dp),
                                              _ptr(kk, _dp), _ptr(sl, _ip), _ptr(ph, _dp), _ptr(idx, _ip),
                                              _ptr(probs, _dp))
    if rc:
        raise ValueError("blossom_oracle_select_pq: bad arguments")
    if G == 1:
        return (idx, probs) if return_scores else idx
    probs = probs.reshape(B, Hkv, G, L, M).sum(axis=2)               # Eq. 12
    gidx = np.full((B, Hkv, L, topk), -1, dtype=np.int32)
    for n in range(B):
        pad0 = 0 if seq_lens is None else L - int(seq_lens[n])
        live = np.array([min((j + 1) * block, L) > max(j * block, pad0) for j in range(M)])
        for g in range(Hkv):
            for t in range(pad0, L):
                b = t // block
                cand = [j for j in range(b) if live[j]]
                best = sorted(cand, key=lambda j: (-probs[n, g, t, j], j))[:topk - 1]
                row = sorted(best) + [b]
                gidx[n, g, t, :len(row)] = row
    return (gidx, probs) if return_scores else gidx


def select_blocks_cmp(q, k, block, topk, cmp_block, cmp_stride, seq_lens=None, sm_scale=None,
                      return_scores=False, phi_logits=None):
    """Eq. 8-11, 13 with overlapping compression blocks (length ``cmp_block``, stride
    ``cmp_stride``) scored and mapped onto selection blocks of ``block`` positions.

    With return_scores also returns the selection scores ``[B,H,M,M]`` and the compression
    scores ``[B,H,M,Mc]``."""
    q, k = _f64(q), _f64(k)
    B, H, L, D = q.shape
    M = -(-L // block)
    if cmp_block < 1 or cmp_stride < 1 or cmp_block % cmp_stride or block % cmp_stride:
        raise ValueError("blossom_oracle_select_cmp: bad arguments")
    Mc = (L - cmp_block) // cmp_stride + 1 if L >= cmp_block else 0
    idx = np.empty((B, H, M, topk), dtype=np.int32)
    scores = np.zeros((B, H, M, M), dtype=np.float64) if return_scores else None
    scores_cmp = np.zeros((B, H, M, max(Mc, 1)), dtype=np.float64) if return_scores else None
    sl = _lens(seq_lens, B)
    if return_scores and Mc == 0:
        sc_arg = None
    else:
        sc_arg = scores_cmp
    ph = _phi(phi_logits, int(cmp_block))
    rc = _load().blossom_oracle_select_cmp(B, H, L, D, block, topk, int(cmp_block), int(cmp_stride),
                                           _scale(sm_scale, D), _ptr(q, _dp), _ptr(k, _dp),
                                           _ptr(sl, _ip), _ptr(ph, _dp), _ptr(idx, _ip), _ptr(scores, _dp),
                                           _ptr(sc_arg, _dp))
    if rc:
        raise ValueError("blossom_oracle_select_cmp: bad arguments")
    if return_scores:
        return idx, scores, scores_cmp[..., :Mc]
    return idx


def forward(q, k, v, gate, block, topk, window, seq_lens=None, sm_scale=None, idx=None,
            stis_mode=0, stis_block=1, per_query=False, gate_mode=0, causal=True):
    """Eq. 14, 16, 17, 19.  ``idx`` overrides the selection when given.

    ``stis_mode`` 0: the short-term branch is the causal window (Eq. 15, first case);
    1: the power-law mask (all of Eq. 15, causal side) with mask block ``stis_block``.

    ``per_query``: the selection is per query position, idx ``[B,H,L,topk]``.
    ``gate_mode`` 1: Eq. 18's input-dependent gate with a one-layer F_o; gate is ``[H, 2 D + 1]`` =
    (w_lt, w_st, b) per head and alpha_t = sigmoid(<w_lt, O_lt,t> + <w_st, O_st,t> + b).
    ``causal=False``: no causal mask (the bidirectional encoders the paper also plugs the
    mechanism into): a query sees every valid key of its selected blocks, and Eq. 15 is symmetric.

    Returns a dict: out, out_lt, out_st ``[B,H,L,D]``, lse ``[2,B,H,L]``, idx.
    """
    q, k, v, gate = _f64(q), _f64(k), _f64(v), _f64(gate)
    B, H, L, D = q.shape
    M = -(-L // block)
    assert gate.shape == ((H, 2 * D + 1) if gate_mode else (H, 2))
    if idx is None:
        if per_query:
            idx = select_blocks_per_query(q, k, block, topk, seq_lens, sm_scale)
        else:
            idx = select_blocks(q, k, block, topk, seq_lens, sm_scale, causal=causal)
    idx = np.ascontiguousarray(np.asarray(idx, dtype=np.int32))
    assert idx.shape == (B, H, L if per_query else M, topk)
    sl = _lens(seq_lens, B)
    out = np.empty_like(q)
    out_lt = np.empty_like(q)
    out_st = np.empty_like(q)
    lse = np.empty((2, B, H, L), dtype=np.float64)
    rc = _load().blossom_oracle_forward(B, H, L, D, block, topk, window, int(stis_mode),
                                        int(stis_block), int(bool(per_query)), int(gate_mode),
                                        int(bool(causal)), _scale(sm_scale, D),
                                        _ptr(q, _dp), _ptr(k, _dp), _ptr(v, _dp), _ptr(gate, _dp),
                                        _ptr(sl, _ip), _ptr(idx, _ip), _ptr(out, _dp),
                                        _ptr(out_lt, _dp), _ptr(out_st, _dp), _ptr(lse, _dp))
    if rc:
        raise ValueError("blossom_oracle_forward: bad arguments")
    return {"out": out, "out_lt": out_lt, "out_st": out_st, "lse": lse, "idx": idx}


def backward(q, k, v, gate, block, topk, window, fwd, dout, seq_lens=None, sm_scale=None,
             stis_mode=0, stis_block=1, per_query=False, gate_mode=0, causal=True):
    """Gradients of sum(out * dout) with the selection frozen.

    ``fwd`` is the dict ``forward`` returned.  Returns dq, dk, dv, dgate (the shape of gate).
    """
    q, k, v, gate, dout = _f64(q), _f64(k), _f64(v), _f64(gate), _f64(dout)
    B, H, L, D = q.shape
    sl = _lens(seq_lens, B)
    idx = np.ascontiguousarray(fwd["idx"], dtype=np.int32)
    out_lt, out_st, lse = _f64(fwd["out_lt"]), _f64(fwd["out_st"]), _f64(fwd["lse"])
    dq, dk, dv = np.empty_like(q), np.empty_like(q), np.empty_like(q)
    dgate = np.empty(gate.shape, dtype=np.float64)
    rc = _load().blossom_oracle_backward(B, H, L, D, block, topk, window, int(stis_mode),
                                         int(stis_block), int(bool(per_query)), int(gate_mode),
                                         int(bool(causal)), _scale(sm_scale, D),
                                         _ptr(q, _dp), _ptr(k, _dp), _ptr(v, _dp),
                                         _ptr(gate, _dp), _ptr(sl, _ip), _ptr(idx, _ip),
                                         _ptr(out_lt, _dp), _ptr(out_st, _dp), _ptr(lse, _dp),
                                         _ptr(dout, _dp), _ptr(dq, _dp), _ptr(dk, _dp),
                                         _ptr(dv, _dp), _ptr(dgate, _dp))
    if rc:
        raise ValueError("blossom_oracle_backward: bad arguments")
    return {"dq": dq, "dk": dk, "dv": dv, "dgate": dgate}


def forward_backward(q, k, v, gate, dout, block, topk, window, seq_lens=None, sm_scale=None,
                     idx=None, stis_mode=0, stis_block=1, per_query=False, gate_mode=0, causal=True):
    """Convenience: forward then backward; returns the two dicts merged."""
    f = forward(q, k, v, gate, block, topk, window, seq_lens, sm_scale, idx, stis_mode, stis_block,
                per_query, gate_mode, causal)
    b = backward(q, k, v, gate, block, topk, window, f, dout, seq_lens, sm_scale, stis_mode,
                 stis_block, per_query, gate_mode, causal)
    f.update(b)
    return f


# ---------------------------------------------------------------------------- rotary positions
# The paper applies RoPE to Q and K before both branches.  Original formulation: the pairs
# (x[2i], x[2i+1]) of a row at position t are rotated by the angle t * theta^(-2i / D).
def _round_to_bf16(x):
    """float64 -> the nearest bfloat16 value (ties to even), returned as float64."""
    x = np.asarray(x, dtype=np.float64)
    f = x.astype(np.float32)
    u = f.view(np.uint32)
    lo = (u & np.uint32(0xFFFF0000)).view(np.float32).astype(np.float64)       # toward zero
    hi = ((u & np.uint32(0xFFFF0000)) + np.uint32(0x10000)).view(np.float32).astype(np.float64)
    dl, dh = np.abs(x - lo), np.abs(hi - x)
    lo_even = ((u >> np.uint32(16)) & np.uint32(1)) == 0
    return np.where((dl < dh) | ((dl == dh) & lo_even), lo, hi)


def rope(x, theta, dtype=None, transpose=False):
    """Rotate ``x [..., L, D]`` by position; ``transpose`` applies the inverse rotation (what the
    chain rule needs for the gradient with respect to the unrotated tensor).  ``dtype`` 'bf16' /
    'fp32' rounds the result once to that storage type; None keeps float64."""
    x = _f64(x)
    L, D = x.shape[-2], x.shape[-1]
    i = np.arange(D // 2, dtype=np.float64)
    ang = np.arange(L, dtype=np.float64)[:, None] * np.power(float(theta), -2.0 * i / D)[None, :]
    if transpose:
        ang = -ang
    cs, sn = np.cos(ang), np.sin(ang)
    out = np.empty_like(x)
    out[..., 0::2] = x[..., 0::2] * cs - x[..., 1::2] * sn
    out[..., 1::2] = x[..., 0::2] * sn + x[..., 1::2] * cs
    if dtype == "bf16":
        return _round_to_bf16(out)
    if dtype == "fp32":
        return out.astype(np.float32).astype(np.float64)
    return out


# ---------------------------------------------------------------------------- grouped-query
# Grouped-query attention: H query heads share Hkv key/value heads, G = H / Hkv query heads per
# group, query head h using key/value head h // G.  The importance scores of the heads of a group
# are summed before the top-k (the paper's group-shared scores, Eq. 12), so a group has one
# selection.  Given the selection every query head is an ordinary head on its group's K and V, so
# the attention and its gradients are the functions above applied to K, V repeated per query head,
# with the K and V gradients of a group's heads summed (the chain rule through the repetition).
def _group(H, Hkv):
    if Hkv < 1 or H % Hkv:
        raise ValueError("heads must be a multiple of kv_heads")
    return H // Hkv


def select_blocks_gqa(q, k, block, topk, seq_lens=None, sm_scale=None, return_scores=False,
                      cmp_block=0, cmp_stride=0, phi_logits=None, causal=True):
    """q ``[B,H,L,D]``, k ``[B,Hkv,L,D]`` -> idx ``[B,Hkv,M,topk]`` from group-summed scores.

    With ``cmp_block`` / ``cmp_stride`` the per-head scores are those of the overlapping
    compression blocks mapped onto the selection blocks (Eq. 8-11); they are then summed over the
    heads of the group (Eq. 12) and the top-k is taken (Eq. 13): the paper's full selection."""
    q, k = _f64(q), _f64(k)
    B, H, L, D = q.shape
    Hkv = k.shape[1]
    G = _group(H, Hkv)
    M = -(-L // block)
    if cmp_block or cmp_stride:
        _, per_head, _ = select_blocks_cmp(q, np.repeat(k, G, axis=1), block, topk, cmp_block or block,
                                           cmp_stride or block, seq_lens, sm_scale, return_scores=True,
                                           phi_logits=phi_logits)
    else:
        _, per_head = select_blocks(q, np.repeat(k, G, axis=1), block, topk, seq_lens, sm_scale,
                                    return_scores=True, phi_logits=phi_logits, causal=causal)
    scores = per_head.reshape(B, Hkv, G, M, M).sum(axis=2)            # Eq. 12
    idx = np.full((B, Hkv, M, topk), -1, dtype=np.int32)
    for n in range(B):
        pad0 = 0 if seq_lens is None else L - int(seq_lens[n])
        live = np.array([min((j + 1) * block, L) > max(j * block, pad0) for j in range(M)])
        for g in range(Hkv):
            for b in range(M):
                if not live[b]:
                    continue
                cand = [j for j in (range(b) if causal else range(M)) if live[j] and j != b]
                # Eq. 13: largest scores first, ties to the lower index; the own block always
                best = sorted(cand, key=lambda j: (-scores[n, g, b, j], j))[:topk - 1]
                row = sorted(best + [b])
                idx[n, g, b, :len(row)] = row
    return (idx, scores) if return_scores else idx


def forward_gqa(q, k, v, gate, block, topk, window, seq_lens=None, sm_scale=None, idx=None,
                cmp_block=0, cmp_stride=0, **kw):
    """``forward`` for q ``[B,H,L,D]`` and k, v ``[B,Hkv,L,D]``; idx is ``[B,Hkv,M,topk]``."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    G = _group(q.shape[1], k.shape[1])
    if idx is None and kw.get("per_query"):
        idx = select_blocks_per_query(q, k, block, topk, seq_lens, sm_scale, cmp_block=cmp_block,
                                      cmp_stride=cmp_stride)
    elif idx is None:
        idx = select_blocks_gqa(q, k, block, topk, seq_lens, sm_scale, cmp_block=cmp_block,
                                cmp_stride=cmp_stride)
    idx = np.ascontiguousarray(np.asarray(idx, dtype=np.int32))
    f = forward(q, np.repeat(k, G, axis=1), np.repeat(v, G, axis=1), gate, block, topk, window,
                seq_lens, sm_scale, idx=np.repeat(idx, G, axis=1), **kw)
    f["idx"] = idx
    return f


def backward_gqa(q, k, v, gate, block, topk, window, fwd, dout, seq_lens=None, sm_scale=None, **kw):
    """``backward`` for grouped heads: dk, dv are ``[B,Hkv,L,D]`` (summed over a group's heads)."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, H, L, D = q.shape
    Hkv = k.shape[1]
    G = _group(H, Hkv)
    f = dict(fwd)
    f["idx"] = np.repeat(np.asarray(fwd["idx"], dtype=np.int32), G, axis=1)
    r = backward(q, np.repeat(k, G, axis=1), np.repeat(v, G, axis=1), gate, block, topk, window, f,
                 dout, seq_lens, sm_scale, **kw)
    r["dk"] = r["dk"].reshape(B, Hkv, G, L, D).sum(axis=2)
    r["dv"] = r["dv"].reshape(B, Hkv, G, L, D).sum(axis=2)
    return r
