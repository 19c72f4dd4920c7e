"""GPU-vs-oracle comparison used by the ``-m gpu`` parity tests.

Tolerances:
  * selected block indices: bit-exact, except rows where the oracle's fp64 scores of the last
    kept and the first dropped candidate differ by < 1e-6 relative;
  * fp32 inputs: max-abs error <= 1e-4 on outputs and gradients;
  * bf16 inputs: max-abs error <= 2e-2 * max|reference| per tensor, never tighter than the fp32
    bar (a tensor whose reference is identically zero, e.g. dq of a one-key softmax, would
    otherwise get a zero tolerance);
  * the log-sum-exps: additionally never looser than 2e-2 ABSOLUTE for bf16 inputs (an error d
    of a log-sum-exp is a relative error e^d - 1 of the softmax normaliser, so bounding it by a
    fraction of max|lse| would let a wrong normaliser through).
When a near-tie row legitimately differs, outputs are compared against the oracle re-run with
the GPU's indices (the attention given the indices is unique).
"""
import numpy as np

import oracle

FP32_ATOL = 1e-4
BF16_REL = 2e-2
TIE_REL = 1e-6
LSE_ATOL = 2e-2


def _grouped(w):
    return bool(w.kv_heads) and w.kv_heads != w.H


def _rotated(w):
    """With rotary positions the library works on q, k rotated and rounded to the storage type."""
    theta = getattr(w, "rope_theta", 0.0)
    if not theta:
        return w
    import copy
    w2 = copy.copy(w)
    w2.q = oracle.rope(w.q, theta, w.dtype)
    w2.k = oracle.rope(w.k, theta, w.dtype)
    w2.rope_theta = 0.0
    return w2


def check_indices(w, gpu_idx, sm_scale=None):
    """Returns the number of forgiven near-tie rows; asserts on any real mismatch."""
    w = _rotated(w)
    pq = bool(getattr(w, "per_query", 0))
    phi = getattr(w, "phi_logits", None)
    if pq:
        ref_idx, scores = oracle.select_blocks_per_query(w.q, w.k, w.block, w.topk, w.seq_lens, sm_scale,
                                                         return_scores=True, phi_logits=phi,
                                                         cmp_block=w.cmp_block, cmp_stride=w.cmp_stride)
    elif _grouped(w):
        ref_idx, scores = oracle.select_blocks_gqa(w.q, w.k, w.block, w.topk, w.seq_lens, sm_scale,
                                                   return_scores=True, cmp_block=w.cmp_block,
                                                   cmp_stride=w.cmp_stride, phi_logits=phi,
                                                   causal=bool(getattr(w, "causal", 1)))
    elif w.cmp_block or w.cmp_stride:
        ref_idx, scores, _ = oracle.select_blocks_cmp(w.q, w.k, w.block, w.topk, w.cmp_block or w.block,
                                                      w.cmp_stride or w.block, w.seq_lens, sm_scale,
                                                      return_scores=True, phi_logits=phi)
    else:
        ref_idx, scores = oracle.select_blocks(w.q, w.k, w.block, w.topk, w.seq_lens, sm_scale,
                                                return_scores=True, phi_logits=phi,
                                                causal=bool(getattr(w, "causal", 1)))
    assert gpu_idx.shape == ref_idx.shape and gpu_idx.dtype == np.int32
    bad = np.argwhere((gpu_idx != ref_idx).any(-1))
    forgiven = 0
    for n, h, b in bad:
        if pq:          # a row per position t (= b here): its candidates are the blocks before t's block
            t, b = b, b // w.block
            S = scores[n, h, t, :b]
            ref_row, gpu_row = ref_idx[n, h, t], gpu_idx[n, h, t]
        else:
            S = scores[n, h, b, :b]
            ref_row, gpu_row = ref_idx[n, h, b], gpu_idx[n, h, b]
        causal = bool(getattr(w, "causal", 1))
        own = b
        cand = np.arange(b) if causal else np.array([j for j in range(scores.shape[-1]) if j != b])
        if not causal:
            S = scores[n, h, b]
        ref_sel = [j for j in ref_row if j >= 0 and j != own]
        gpu_sel = [j for j in gpu_row if j >= 0 and j != own]
        # structure must still be valid
        g = [int(j) for j in gpu_row if j >= 0]
        assert g == sorted(set(g)) and own in g and len(g) == len(ref_sel) + 1, (n, h, b, g)
        if causal:
            assert g[-1] == own
        dropped = np.setdiff1d(cand, ref_sel)
        kept_min = S[ref_sel].min()
        drop_max = S[dropped].max()
        gap = abs(kept_min - drop_max) / max(abs(kept_min), abs(drop_max))
        assert gap < TIE_REL, f"selection mismatch at {(n, h, b)}: ref {ref_sel} gpu {gpu_sel} gap {gap:.3e}"
        # the GPU may only have swapped candidates inside the tie
        for j in np.setxor1d(ref_sel, gpu_sel):
            assert abs(S[j] - kept_min) / abs(kept_min) < TIE_REL
        forgiven += 1
    return forgiven


def tolerance(w, ref):
    if w.dtype == "fp32":
        return FP32_ATOL
    return max(BF16_REL * float(np.abs(ref).max()), FP32_ATOL)


def check_forward_backward(w, res, sm_scale=None, backward=True):
    """res: dict of numpy arrays from the CUDA path.  Returns a dict of max-abs errors."""
    theta = getattr(w, "rope_theta", 0.0)
    w = _rotated(w)
    forgiven = check_indices(w, res["idx"], sm_scale)
    fwd_fn, bwd_fn = (oracle.forward_gqa, oracle.backward_gqa) if _grouped(w) else (oracle.forward, oracle.backward)
    kw = {"per_query": True} if getattr(w, "per_query", 0) else {}
    if getattr(w, "gate_mode", 0):
        kw["gate_mode"] = 1
    if not getattr(w, "causal", 1):
        kw["causal"] = False
    ref = fwd_fn(w.q, w.k, w.v, w.gate, w.block, w.topk, w.window, w.seq_lens, sm_scale,
                 idx=res["idx"], stis_mode=w.stis_mode, stis_block=w.stis_block, **kw)
    errs = {"near_tie_rows": forgiven}
    keys = ["out", "out_lt", "out_st", "lse"]
    if backward:
        ref.update(bwd_fn(w.q, w.k, w.v, w.gate, w.block, w.topk, w.window, ref, w.dout,
                          w.seq_lens, sm_scale, stis_mode=w.stis_mode, stis_block=w.stis_block, **kw))
        if theta:   # gradients with respect to the unrotated q, k: the transpose of the rotation
            ref["dq"] = oracle.rope(ref["dq"], theta, transpose=True)
            ref["dk"] = oracle.rope(ref["dk"], theta, transpose=True)
        keys += ["dq", "dk", "dv", "dgate"]
    for key in keys:
        if res.get(key) is None:
            continue
        got = np.asarray(res[key], dtype=np.float64)
        assert np.isfinite(got).all(), f"{key}: non-finite values"
        err = float(np.abs(got - ref[key]).max())
        tol = tolerance(w, ref[key])
        if key == "lse":
            tol = min(tol, LSE_ATOL) if w.dtype != "fp32" else tol
        errs[key] = err
        assert err <= tol, f"{w.name} {key}: max-abs error {err:.3e} > tol {tol:.3e}"
    return errs
