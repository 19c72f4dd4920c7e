"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, sizes workspaces, names its statuses and rejects bad arguments before any launch."""
import ctypes
import os
import re

import pytest

from paper_2512_13368_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def header_functions():
    text = open(os.path.join(ROOT, "include", "blossom.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(blossom_[a-z_]+)\s*\(", text)))


def test_exports_match_header(lib):
    names = header_functions()
    assert set(names) == set(binding.EXPORTS), names
    for n in names:
        assert getattr(lib, n) is not None


def test_version_and_status_strings(lib):
    assert binding.blossom_version() >= 100
    seen = {binding.blossom_status_string(i) for i in range(6)}
    assert len(seen) == 6 and "ok" in seen
    assert binding.blossom_status_string(99) == "unknown status"


def good(**kw):
    d = dict(batch=4, heads=2, seq_len=64, head_dim=32, block_size=8, top_k=2, window=16, dtype="fp32")
    d.update(kw)
    return binding.make_params(**d)


def test_workspace_bytes(lib):
    n = binding.blossom_workspace_bytes(good())
    assert n > 0 and n % 256 == 0
    assert binding.blossom_workspace_bytes(good(batch=8)) > n
    for bad in (dict(batch=0), dict(head_dim=48), dict(block_size=12), dict(top_k=0), dict(window=0),
                dict(kv_heads=3), dict(kv_heads=0), dict(kv_strides=(4096, 2048, 31)), dict(causal=2), dict(causal=0, select_mode=1), dict(select_mode=2), dict(select_mode=1, cmp_block=16, cmp_stride=4, seq_len=2048), dict(dtype=7),
                dict(seq_len=8 * 1025), dict(strides=(4096, 2048, 33)), dict(sm_scale=-1.0),
                dict(stis_mode=2), dict(stis_mode=-1), dict(stis_mode=1, stis_block=-3),
                dict(cmp_block=12, cmp_stride=8), dict(cmp_block=16, cmp_stride=3), dict(cmp_block=-8)):
        assert binding.blossom_workspace_bytes(good(**bad)) == 0, bad
    assert binding.blossom_workspace_bytes(good(stis_mode=1, stis_block=4)) == n  # power-law mask
    assert binding.blossom_workspace_bytes(good(cmp_block=8, cmp_stride=8)) == n    # same as the default
    assert binding.blossom_workspace_bytes(good(cmp_block=16, cmp_stride=4)) > n    # overlapping blocks
    assert binding.blossom_workspace_bytes(good(kv_heads=1)) == n                   # grouped key/value heads


def test_argument_validation_precedes_any_launch(lib):
    p = good()
    A = 1 << 20  # a fake, aligned, never-dereferenced device address
    ws_bytes = binding.blossom_workspace_bytes(p)
    E = binding
    # NULL tensors
    assert E.blossom_attn_fwd(p, None, A, A, A, None, A, 0, A, A, A, A, A, ws_bytes, stream=0, check=False) == E.BLOSSOM_ERR_INVALID_ARG
    # misaligned q
    assert E.blossom_attn_fwd(p, A + 4, A, A, A, None, A, 0, A, A, A, A, A, ws_bytes, stream=0, check=False) == E.BLOSSOM_ERR_INVALID_ARG
    # only one of the saved outputs
    assert E.blossom_attn_fwd(p, A, A, A, A, None, A, 0, A, A, None, A, A, ws_bytes, stream=0, check=False) == E.BLOSSOM_ERR_INVALID_ARG
    # training outputs without lse
    assert E.blossom_attn_fwd(p, A, A, A, A, None, A, 0, A, A, A, None, A, ws_bytes, stream=0, check=False) == E.BLOSSOM_ERR_INVALID_ARG
    # workspace: missing, misaligned, short
    assert E.blossom_attn_fwd(p, A, A, A, A, None, A, 0, A, A, A, A, None, 0, stream=0, check=False) == E.BLOSSOM_ERR_WORKSPACE
    assert E.blossom_attn_fwd(p, A, A, A, A, None, A, 0, A, A, A, A, A + 64, ws_bytes, stream=0, check=False) == E.BLOSSOM_ERR_WORKSPACE
    assert E.blossom_attn_fwd(p, A, A, A, A, None, A, 0, A, A, A, A, A, ws_bytes - 1, stream=0, check=False) == E.BLOSSOM_ERR_WORKSPACE
    # unsupported but legal requests
    assert E.blossom_attn_fwd(good(select_mode=1, cmp_block=16, cmp_stride=4, seq_len=2048), A, A, A, A, None, A, 0, A, A, A, A, A, ws_bytes, stream=0, check=False) == E.BLOSSOM_ERR_UNSUPPORTED
    assert E.blossom_attn_fwd(good(kv_heads=3), A, A, A, A, None, A, 0, A, A, A, A, A, ws_bytes, stream=0, check=False) == E.BLOSSOM_ERR_INVALID_ARG
    assert E.blossom_select_blocks(good(head_dim=128), A, A, None, A, A, ws_bytes, stream=0, check=False) == E.BLOSSOM_ERR_UNSUPPORTED
    # one block more than the 1024 the lists are laid out for
    big = good(seq_len=1024 * 16 + 1, block_size=16)
    assert E.blossom_select_blocks(big, A, A, None, A, A, 1 << 40, stream=0, check=False) == E.BLOSSOM_ERR_UNSUPPORTED
    assert E.blossom_select_blocks(p, A, None, None, A, A, ws_bytes, stream=0, check=False) == E.BLOSSOM_ERR_INVALID_ARG
    # backward: every tensor is required
    args = [A] * 14          # q k v gate seq_lens idx out_lt out_st lse dout dq dk dv dgate
    for i in (0, 3, 5, 6, 8, 9, 10, 13):
        a = list(args)
        a[i] = None
        a[4] = None              # seq_lens may always be NULL
        assert E.blossom_attn_bwd(p, *a, A, ws_bytes, stream=0, check=False) == E.BLOSSOM_ERR_INVALID_ARG, i
    with pytest.raises(E.BlossomError):
        E.blossom_select_blocks(p, None, None, None, None, None, 0, stream=0)


def test_params_struct_layout_matches_header():
    # 12 x 4-byte fields, three int64 strides, the two short-term mask fields, the two
    # compression-block fields, three int64 key/value strides and the pointer to the summary
    # logits, the gate mode, the rotary base, the tile-list promise: 136 bytes with natural alignment
    assert ctypes.sizeof(binding.blossom_params) == 136
    assert binding.blossom_params.phi_logits.offset == 112 and binding.blossom_params.gate_mode.offset == 120
    assert binding.blossom_params.kv_stride_b.offset == 88
    assert binding.blossom_params.cmp_block.offset == 80 and binding.blossom_params.cmp_stride.offset == 84
    assert binding.blossom_params.stride_b.offset == 48
    assert binding.blossom_params.stis_mode.offset == 72 and binding.blossom_params.stis_block.offset == 76


# ---- the autograd front end validates what it hands to the library as raw addresses -------------
def _qkv(B=2, H=4, L=16, D=32, Hkv=None, dtype=None):
    import torch
    dtype = dtype or torch.bfloat16
    q = torch.zeros(B, H, L, D, dtype=dtype)
    k = torch.zeros(B, Hkv or H, L, D, dtype=dtype)
    return q, k, k.clone()


def test_autograd_front_end_rejects_bad_arguments_before_any_launch():
    import torch
    from paper_2512_13368_b200.autograd import check_arguments
    q, k, v = _qkv()
    gate = torch.zeros(4, 2)
    with pytest.raises(ValueError):           # host tensors: the library would dereference host addresses
        check_arguments(q, k, v, gate, None)
    chk = lambda *a: check_arguments(*a, require_cuda=False)  # noqa: E731
    assert chk(q, k, v, gate, None) is None
    with pytest.raises(ValueError):
        chk(q, k, v, torch.zeros(4, 3), None)                 # gate shape
    with pytest.raises(ValueError):
        chk(q, k, v, torch.zeros(2, 2), None)
    with pytest.raises(TypeError):
        chk(q, k, v, torch.zeros(4, 2, dtype=torch.int32), None)
    with pytest.raises(ValueError):
        chk(q, k, v, gate.to("meta"), None)                   # another device
    with pytest.raises(ValueError):
        chk(q, k, v, gate, torch.zeros(3, dtype=torch.int32))  # wrong number of lengths
    with pytest.raises(TypeError):
        chk(q, k, v, gate, torch.zeros(2, dtype=torch.float32))
    with pytest.raises(ValueError):
        chk(q, k, v, gate, torch.zeros(2, dtype=torch.int32, device="meta"))
    lens = chk(q, k, v, gate, torch.tensor([16, 3], dtype=torch.int64))
    assert lens.dtype == torch.int32 and lens.tolist() == [16, 3]   # int64 would be read as int32 pairs
    with pytest.raises(TypeError):
        chk(q, k.float(), v.float(), gate, None)
    with pytest.raises(ValueError):
        chk(q, *_qkv(Hkv=3)[1:], gate, None)                  # 4 heads on 3 key/value heads
    q2, k2, v2 = _qkv(Hkv=2)
    assert chk(q2, k2, v2, gate, None) is None                # grouped heads


def test_every_q_shaped_buffer_gets_q_strides():
    import torch
    from paper_2512_13368_b200.autograd import _dense, _like
    qkv = torch.zeros(2, 16, 3, 4, 32)                        # packed projection [B, L, 3, H, D]
    q = qkv[:, :, 0].permute(0, 2, 1, 3)                      # [B, H, L, D], equal strides, not dense
    assert not _dense(q)
    assert torch.empty_like(q).stride() != q.stride()         # what made the library overrun its outputs
    assert _like(q).stride() == q.stride()
    qc = q.contiguous()
    assert _dense(qc) and _like(qc).stride() == qc.stride()
    perm = torch.zeros(2, 16, 4, 32).permute(0, 2, 1, 3)      # [B, L, H, D] storage: dense, kept as is
    assert _dense(perm) and _like(perm).stride() == perm.stride()


def test_debug_switch_arguments(lib):
    assert lib.blossom_debug_switch(0, -1) == 0 and lib.blossom_debug_switch(1, -1) == 0
    assert lib.blossom_debug_switch(2, -1) == 0
    assert lib.blossom_debug_switch(3, 0) == binding.BLOSSOM_ERR_INVALID_ARG
    assert lib.blossom_debug_switch(0, 2) == binding.BLOSSOM_ERR_INVALID_ARG


def test_static_selection_rejects_overlapping_compression_blocks(lib):
    A = 1 << 20
    prm = good(cmp_block=16, cmp_stride=4)
    rc = binding.blossom_select_blocks_static(prm, A, A, None, A, stream=0, check=False)
    assert rc == binding.BLOSSOM_ERR_UNSUPPORTED
