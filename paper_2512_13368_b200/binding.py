"""ctypes binding of ``libblossom.so`` (the C ABI declared in ``include/blossom.h``).

Argument marshalling only: every step of the path runs in the CUDA library.  Functions keep
the C names.  Tensor arguments may be ``torch.Tensor`` (their ``data_ptr()`` is passed), an
``int`` address, or ``None`` (NULL).  A non-zero status raises ``BlossomError``.  There is no
fallback: if the shared library is missing the first call raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libblossom.so")

BLOSSOM_OK = 0
BLOSSOM_ERR_INVALID_ARG = 1
BLOSSOM_ERR_UNSUPPORTED = 2
BLOSSOM_ERR_WORKSPACE = 3
BLOSSOM_ERR_CUDA = 4
BLOSSOM_ERR_TIMEOUT = 5
BLOSSOM_ERR_TOO_LARGE = 6
DTYPE_FP32 = 0
DTYPE_BF16 = 1

EXPORTS = (
    "blossom_workspace_bytes", "blossom_select_blocks", "blossom_select_blocks_static",
    "blossom_attn_fwd", "blossom_attn_bwd",
    "blossom_device_status", "blossom_status_string", "blossom_version", "blossom_launch_count",
    "blossom_profile_start", "blossom_profile_every", "blossom_profile_stop", "blossom_kernel_name",
    "blossom_debug_switch",
    "blossom_selftest_wait_timeout",
)


class blossom_params(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("heads", ctypes.c_int32), ("kv_heads", ctypes.c_int32),
        ("seq_len", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("block_size", ctypes.c_int32),
        ("top_k", ctypes.c_int32), ("window", ctypes.c_int32), ("causal", ctypes.c_int32),
        ("select_mode", ctypes.c_int32), ("dtype", ctypes.c_int32), ("sm_scale", ctypes.c_float),
        ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_l", ctypes.c_int64),
        ("stis_mode", ctypes.c_int32), ("stis_block", ctypes.c_int32),
        ("cmp_block", ctypes.c_int32), ("cmp_stride", ctypes.c_int32),
        ("kv_stride_b", ctypes.c_int64), ("kv_stride_h", ctypes.c_int64), ("kv_stride_l", ctypes.c_int64),
        ("phi_logits", ctypes.c_void_p), ("gate_mode", ctypes.c_int32),
        ("rope_theta", ctypes.c_float),
        ("reuse_tile_lists", ctypes.c_int32),
    ]


class BlossomError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__(f"{where}: {blossom_status_string(status)} (status {int(status)})")


_lib = None


def load():
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2512_13368_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    pp = ctypes.POINTER(blossom_params)
    lib.blossom_workspace_bytes.restype = sz
    lib.blossom_workspace_bytes.argtypes = [pp]
    lib.blossom_select_blocks.restype = ctypes.c_int
    lib.blossom_select_blocks.argtypes = [pp, vp, vp, vp, vp, vp, sz, vp]
    lib.blossom_select_blocks_static.restype = ctypes.c_int
    lib.blossom_select_blocks_static.argtypes = [pp, vp, vp, vp, vp, vp]
    lib.blossom_attn_fwd.restype = ctypes.c_int
    lib.blossom_attn_fwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp]
    lib.blossom_attn_bwd.restype = ctypes.c_int
    lib.blossom_attn_bwd.argtypes = [pp] + [vp] * 15 + [sz, vp]
    lib.blossom_device_status.restype = ctypes.c_int
    lib.blossom_device_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.blossom_status_string.restype = ctypes.c_char_p
    lib.blossom_status_string.argtypes = [ctypes.c_int]
    lib.blossom_version.restype = ctypes.c_int
    lib.blossom_launch_count.restype = ctypes.c_uint64
    lib.blossom_profile_start.restype = ctypes.c_int
    lib.blossom_profile_start.argtypes = [ctypes.c_int]
    lib.blossom_profile_every.restype = ctypes.c_int
    lib.blossom_profile_every.argtypes = [ctypes.c_int]
    lib.blossom_profile_stop.restype = ctypes.c_int
    lib.blossom_profile_stop.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_float), ctypes.c_int]
    lib.blossom_kernel_name.restype = ctypes.c_char_p
    lib.blossom_kernel_name.argtypes = [ctypes.c_int]
    lib.blossom_selftest_wait_timeout.restype = ctypes.c_int
    lib.blossom_selftest_wait_timeout.argtypes = [vp, sz, vp]
    lib.blossom_debug_switch.restype = ctypes.c_int
    lib.blossom_debug_switch.argtypes = [ctypes.c_int, ctypes.c_int]
    _lib = lib
    return lib


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _nbytes(x):
    if isinstance(x, int):
        return x
    return x.numel() * x.element_size()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def make_params(batch, heads, seq_len, head_dim, block_size, top_k, window, dtype, sm_scale=0.0,
                strides=None, kv_heads=None, causal=1, select_mode=0, stis_mode=0,
                stis_block=1, cmp_block=0, cmp_stride=0, kv_strides=None, phi_logits=None,
                gate_mode=0, rope_theta=0.0, reuse_tile_lists=0) -> blossom_params:
    """Fill a ``blossom_params``; ``strides`` = (stride_b, stride_h, stride_l) in elements,
    default contiguous [B, H, L, D].  ``phi_logits``: float32 device tensor (the caller keeps it
    alive) or None."""
    if strides is None:
        strides = (heads * seq_len * head_dim, seq_len * head_dim, head_dim)
    d = {"fp32": DTYPE_FP32, "bf16": DTYPE_BF16}.get(dtype, dtype)
    return blossom_params(batch, heads, heads if kv_heads is None else kv_heads, seq_len, head_dim,
                          block_size, top_k, window, causal, select_mode, d, float(sm_scale),
                          int(strides[0]), int(strides[1]), int(strides[2]), int(stis_mode),
                          int(stis_block), int(cmp_block), int(cmp_stride),
                          *((0, 0, 0) if kv_strides is None else [int(x) for x in kv_strides]),
                          _ptr(phi_logits), int(gate_mode), float(rope_theta), int(reuse_tile_lists))


def blossom_status_string(status) -> str:
    return load().blossom_status_string(int(status)).decode()


def blossom_version() -> int:
    return int(load().blossom_version())


def blossom_launch_count() -> int:
    return int(load().blossom_launch_count())


def blossom_workspace_bytes(params) -> int:
    return int(load().blossom_workspace_bytes(ctypes.byref(params)))


def blossom_select_blocks(params, q, k, seq_lens, block_idx, workspace, workspace_bytes=None,
                          stream=None, check=True) -> int:
    rc = load().blossom_select_blocks(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(seq_lens),
                                      _ptr(block_idx), _ptr(workspace),
                                      _nbytes(workspace) if workspace_bytes is None else workspace_bytes,
                                      _stream(stream))
    if rc and check:
        raise BlossomError(rc, "blossom_select_blocks")
    return rc


def blossom_select_blocks_static(params, q, k, seq_lens, block_idx, stream=None, check=True) -> int:
    """Selection without a caller workspace: the scratch is a fixed array inside the library, so
    nothing on the path allocates.  For callers that are handed tensors but may not allocate
    device memory themselves.  Capacity-limited (see include/blossom.h); calls that could overlap
    on one device must be serialised by the caller."""
    rc = load().blossom_select_blocks_static(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(seq_lens),
                                             _ptr(block_idx), _stream(stream))
    if rc and check:
        raise BlossomError(rc, "blossom_select_blocks_static")
    return rc


def blossom_attn_fwd(params, q, k, v, gate_logits, seq_lens, block_idx, idx_is_input, out, out_lt,
                     out_st, lse, workspace, workspace_bytes=None, stream=None, check=True) -> int:
    rc = load().blossom_attn_fwd(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(gate_logits),
                                 _ptr(seq_lens), _ptr(block_idx), int(idx_is_input), _ptr(out),
                                 _ptr(out_lt), _ptr(out_st), _ptr(lse), _ptr(workspace),
                                 _nbytes(workspace) if workspace_bytes is None else workspace_bytes,
                                 _stream(stream))
    if rc and check:
        raise BlossomError(rc, "blossom_attn_fwd")
    return rc


def blossom_attn_bwd(params, q, k, v, gate_logits, seq_lens, block_idx, out_lt, out_st, lse, dout,
                     dq, dk, dv, dgate, workspace, workspace_bytes=None, stream=None,
                     check=True) -> int:
    rc = load().blossom_attn_bwd(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(gate_logits),
                                 _ptr(seq_lens), _ptr(block_idx), _ptr(out_lt), _ptr(out_st),
                                 _ptr(lse), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dgate),
                                 _ptr(workspace),
                                 _nbytes(workspace) if workspace_bytes is None else workspace_bytes,
                                 _stream(stream))
    if rc and check:
        raise BlossomError(rc, "blossom_attn_bwd")
    return rc


def blossom_device_status(workspace, stream=None) -> int:
    out = ctypes.c_int32(-1)
    rc = load().blossom_device_status(_ptr(workspace), _stream(stream), ctypes.byref(out))
    if rc:
        raise BlossomError(rc, "blossom_device_status")
    return int(out.value)


def blossom_profile_start(max_launches: int) -> None:
    rc = load().blossom_profile_start(int(max_launches))
    if rc:
        raise BlossomError(rc, "blossom_profile_start")


def blossom_profile_every(n: int) -> None:
    rc = load().blossom_profile_every(int(n))
    if rc:
        raise BlossomError(rc, "blossom_profile_every")


def blossom_profile_stop(capacity: int):
    """Returns a list of (kernel name, milliseconds), one entry per recorded launch."""
    ids = (ctypes.c_int32 * capacity)()
    ms = (ctypes.c_float * capacity)()
    n = load().blossom_profile_stop(ids, ms, int(capacity))
    if n < 0:
        raise RuntimeError("blossom_profile_stop failed (no profile running or a CUDA error)")
    return [(blossom_kernel_name(ids[i]), float(ms[i])) for i in range(n)]


def blossom_kernel_name(kernel_id: int) -> str:
    return load().blossom_kernel_name(int(kernel_id)).decode()


SWITCH_FORCE_SIMT = 0
SWITCH_EXACT_SELECT = 1
SWITCH_SERIAL_LAUNCH = 2


def blossom_debug_switch(which: int, value: int) -> None:
    """Process-wide debugging switch: 1 on, 0 off, -1 back to the environment's default."""
    rc = load().blossom_debug_switch(int(which), int(value))
    if rc:
        raise BlossomError(rc, "blossom_debug_switch")


def blossom_selftest_wait_timeout(workspace, stream=None) -> None:
    """Launch the diagnostic kernel whose only wait cannot complete; read the outcome with
    ``blossom_device_status(workspace)`` (it must be BLOSSOM_ERR_TIMEOUT)."""
    rc = load().blossom_selftest_wait_timeout(_ptr(workspace), _nbytes(workspace), _stream(stream))
    if rc:
        raise BlossomError(rc, "blossom_selftest_wait_timeout")
