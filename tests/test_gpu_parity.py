"""Parity of the CUDA library (through its C ABI) against the fp64 oracle on the same seeded
inputs.  Every test here needs a B200."""
import numpy as np
import pytest

from paper_2512_13368_b200 import workloads
from parity_util import check_forward_backward, check_indices, tolerance

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def runner():
    import torch
    assert torch.cuda.is_available(), "the gpu-marked tests need a CUDA device"
    from paper_2512_13368_b200 import binding, runner
    binding.load()  # fail loudly if the extension is missing
    return runner


def run(runner, w, sm_scale=0.0, training=True, backward=True):
    p = runner.DeviceProblem(w, sm_scale=sm_scale, training=training)
    p.forward()
    if backward:
        p.backward()
    from paper_2512_13368_b200 import binding
    assert binding.blossom_device_status(p.workspace) == 0
    return p, p.results()


# ----------------------------------------------------------------- element-by-element cases
def test_config1_tiny_fp32(runner):
    w = workloads.config1()
    _, res = run(runner, w)
    errs = check_forward_backward(w, res)
    print(errs)


@pytest.mark.parametrize("B", [24])
def test_config2_padded_bf16(runner, B):
    w = workloads.config2(B=B)         # 24 sequences: lengths 5..200, ragged last block of 8 rows
    _, res = run(runner, w)
    errs = check_forward_backward(w, res)
    print(errs)
    # padded rows are exactly zero everywhere
    for n in range(w.B):
        pad0 = w.L - int(w.seq_lens[n])
        for key in ("out", "out_lt", "out_st", "dq", "dk", "dv"):
            assert np.all(res[key][n, :, :pad0] == 0.0)
        assert np.all(res["lse"][:, n, :, :pad0] == 0.0)


def test_config3_mid_reduced_batch(runner):
    w = workloads.config3(B=2)
    _, res = run(runner, w)
    print(check_forward_backward(w, res))


def test_config4_long_reduced_batch(runner):
    w = workloads.config4(B=1)          # 8 heads x L4096: several tiles + every block count
    _, res = run(runner, w)
    print(check_forward_backward(w, res))


def test_config5_attention_shape(runner):
    w = workloads.config5_attention(B=2)
    _, res = run(runner, w)
    print(check_forward_backward(w, res))


# ---------------------------------------------------------------------------- edge cases
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("L,D,block,topk,window,lens", [
    (1, 32, 8, 1, 1, None),              # one token
    (7, 32, 8, 4, 3, None),              # shorter than one block
    (200, 32, 16, 4, 32, [200, 5, 1, 0]),  # ragged tail, length-1 and fully padded sequences
    (130, 64, 64, 16, 256, [130, 66]),   # top-k and window larger than the sequence
    (96, 64, 32, 8, 200, None),          # window > L  (short-term branch = dense)
    (257, 64, 8, 5, 9, [257, 100]),      # many small blocks, odd length
    (192, 32, 64, 2, 1, None),           # window 1: short-term branch returns v
    (512, 64, 64, 64, 64, None),         # top-k covers every block (long-term branch = dense)
    (1000, 64, 32, 6, 100, [1000, 333]),   # several 128-row tiles, ragged last tile, padding inside a tile
    (700, 32, 16, 9, 48, [700, 129, 64]),  # two query blocks per warp, padding ends on a tile border
    (384, 64, 16, 3, 130, None),           # window wider than two tiles, few selected blocks
])
def test_edge_shapes(runner, dtype, L, D, block, topk, window, lens):
    B = len(lens) if lens else 2
    w = workloads.make("edge", dtype, B, 2, L, D, block, topk, window, seed=11)
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    _, res = run(runner, w)
    print(check_forward_backward(w, res))


@pytest.mark.gpu
@pytest.mark.parametrize("D,topk,window,lens", [(32, 8, 128, None), (64, 4, 64, [65536 - 4097])])
def test_maximum_number_of_blocks(runner, D, topk, window, lens):
    """ceil(L / block) = 1024, the most the interface takes: 1024 entries on every tile list, 512
    CTAs per unit, query blocks with more than a thousand candidates in the selection."""
    w = workloads.make("max-blocks", "bf16", 1, 2, 65536, D, 64, topk, window, seed=23)
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    _, res = run(runner, w)
    print(check_forward_backward(w, res))


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("L,D,block,topk,window,blk,lens", [
    (64, 32, 8, 2, 8, 1, None),              # the paper's defaults: window 8, mask block 1
    (200, 32, 16, 4, 8, 1, [200, 5, 1, 0]),  # ragged tail, length-1 and fully padded sequences
    (300, 64, 32, 4, 16, 4, [300, 131]),     # mask block 4: whole blocks at power-of-two distances
    (257, 64, 8, 5, 3, 2, None),             # window not a multiple of the mask block, odd length
    (96, 64, 64, 2, 200, 1, None),           # window > L: the mask adds nothing to dense causal
    (128, 32, 16, 3, 1, 128, None),          # mask block = L: every key is in the last block
    (1024, 64, 64, 8, 8, 1, [1024, 700]),    # links up to distance 512 across many key blocks
])
def test_power_law_short_term_mask(runner, dtype, L, D, block, topk, window, blk, lens):
    """Eq. 15 with all three cases (stis_mode 1) against the oracle, forward and backward."""
    B = len(lens) if lens else 2
    w = workloads.make("powerlaw", dtype, B, 2, L, D, block, topk, window, seed=13, stis_mode=1,
                       stis_block=blk)
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    _, res = run(runner, w)
    print(check_forward_backward(w, res))


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("L,D,block,topk,l,s,lens,power_law", [
    (256, 32, 16, 4, 32, 16, None, True),            # the paper's default sizes, with its short-term mask
    (512, 64, 16, 4, 32, 16, [512, 200, 33], False),
    (320, 64, 32, 3, 32, 16, [320, 150], False),     # two strides per selection block
    (192, 32, 16, 5, 48, 8, None, False),            # long compression blocks, small stride
    (20, 32, 16, 4, 32, 16, None, False),            # shorter than one compression block
    (1024, 64, 64, 8, 128, 32, [1024, 611], False),  # tensor-core attention behind the new selection
])
def test_overlapping_compression_blocks(runner, dtype, L, D, block, topk, l, s, lens, power_law):
    """Selection through overlapping compression blocks and the score remap (Eq. 8-11)."""
    B = len(lens) if lens else 2
    w = workloads.make("overlap", dtype, B, 2, L, D, block, topk, 8 if power_law else 24, seed=17,
                       stis_mode=1 if power_law else 0)
    w.cmp_block, w.cmp_stride = l, s
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    _, res = run(runner, w)
    print(check_forward_backward(w, res))


@pytest.mark.gpu
def test_input_dependent_gate_runs_on_the_tensor_core_kernels(runner):
    """bf16 shapes the tensor-core kernels take keep them with gate_mode 1 (one forward kernel plus
    a row-wise mix; one backward pass per branch plus an addition): the launch record shows those
    kernels, the results agree with the oracle and with the CUDA-core path, and a forward call
    that returns no branch outputs gives the same output bits."""
    from paper_2512_13368_b200 import binding
    w = workloads.make("gate-tc", "bf16", 3, 4, 1000, 64, 32, 6, 70, seed=71, kv_heads=2, lengths=(300, 1000))
    w.gate_mode = 1
    w.gate = (0.3 * np.random.default_rng(6).standard_normal((w.H, 2 * w.D + 1))).astype(np.float32)
    binding.blossom_profile_start(64)
    _, tc = run(runner, w)
    names = {name for name, _ in binding.blossom_profile_stop(64)}
    assert {"fwd_tc", "bwd_dq_tc", "bwd_dkdv_tc"} <= names and not any("simt" in x for x in names), names
    print(check_forward_backward(w, tc))
    q, _ = run(runner, w, training=False, backward=False)
    assert np.array_equal(q.results()["out"], tc["out"])
    binding.blossom_debug_switch(binding.SWITCH_FORCE_SIMT, 1)
    try:
        _, simt = run(runner, w)
    finally:
        binding.blossom_debug_switch(binding.SWITCH_FORCE_SIMT, -1)
    for key in ("out", "out_lt", "out_st", "lse", "dq", "dk", "dv", "dgate"):
        ref = np.abs(simt[key]).max()
        err = np.abs(tc[key] - simt[key]).max()
        assert err <= 2e-2 * max(ref, 1e-3), (key, err, ref)


def test_config4_full_size_input_dependent_gate(runner):
    """The headline shape with Eq. 18's gate, as the benchmark's --input-gate option times it."""
    w = workloads.config4()
    w.gate_mode = 1
    w.gate = (np.random.default_rng(1004).standard_normal((w.H, 2 * w.D + 1)) / np.sqrt(w.D)).astype(np.float32)
    errs, res = _whole_batch(runner, w)
    print(errs)
    assert res["dgate"].shape == (w.H, 2 * w.D + 1)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("L,D,H,Hkv,block,topk,window,lens,power_law", [
    (64, 32, 4, 2, 8, 2, 16, None, False),
    (200, 32, 8, 2, 16, 4, 32, [200, 5, 77], False),     # the paper's 8 heads on 2 key/value heads, padded
    (300, 64, 6, 3, 32, 4, 40, [300, 131], False),
    (256, 64, 4, 1, 64, 3, 8, None, True),               # one key/value head, power-law short-term mask
    (1024, 64, 8, 2, 64, 8, 256, [1024, 640], False),
    (448, 64, 6, 2, 32, 4, 40, [448, 131], False),       # an odd number of heads per key/value head
    (330, 32, 4, 2, 16, 3, 24, [330, 9, 200], True),     # pairs of heads, six 64-position tiles, the last ragged
    (577, 64, 4, 2, 64, 5, 100, [577, 64, 65], False),   # pairs of heads, an odd number of tiles
])
def test_grouped_query_heads(runner, dtype, L, D, H, Hkv, block, topk, window, lens, power_law):
    """Query heads share key/value heads and one selection per group (summed scores, Eq. 12)."""
    B = len(lens) if lens else 2
    w = workloads.make("gqa", dtype, B, H, L, D, block, topk, window, seed=19, kv_heads=Hkv,
                       stis_mode=1 if power_law else 0)
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    _, res = run(runner, w)
    assert res["dk"].shape == (B, Hkv, L, D) and res["idx"].shape[1] == Hkv
    print(check_forward_backward(w, res))


@pytest.mark.parametrize("dtype,D", [("fp32", 32), ("bf16", 32), ("bf16", 64)])
def test_paper_default_configuration_in_one_call(runner, dtype, D):
    """The configuration the paper evaluates, all in one call: 8 query heads on 2 key/value heads
    with one selection per group (Eq. 12), compression blocks of 32 at stride 16 scored and mapped
    onto selection blocks of 16 (Eq. 8-11), top-4, and the power-law short-term mask with window 8
    and mask block 1 (Eq. 15), at the paper's sequence length 200 with left padding."""
    w = workloads.make("paper-default", dtype, 5, 8, 200, D, 16, 4, 8, seed=29, std=0.7, kv_heads=2,
                       stis_mode=1, stis_block=1)
    w.cmp_block, w.cmp_stride = 32, 16
    w.seq_lens = np.asarray([200, 131, 33, 16, 0], dtype=np.int32)
    _, res = run(runner, w)
    assert res["idx"].shape == (5, 2, 13, 4) and res["dk"].shape == (5, 2, 200, D)
    print(check_forward_backward(w, res))


@pytest.mark.parametrize("dtype,D", [("fp32", 32), ("bf16", 32), ("bf16", 64)])
def test_paper_default_configuration_with_its_selection_per_query_position(runner, dtype, D):
    """The same configuration with the selection as the paper prints it (Eq. 13 per query
    position, through the compression blocks and Eq. 11, shared by the heads of a group)."""
    w = workloads.make("paper-exact", dtype, 5, 8, 200, D, 16, 4, 8, seed=37, std=0.7, kv_heads=2,
                       stis_mode=1, stis_block=1)
    w.cmp_block, w.cmp_stride, w.per_query = 32, 16, 1
    w.seq_lens = np.asarray([200, 131, 33, 16, 0], dtype=np.int32)
    _, res = run(runner, w)
    assert res["idx"].shape == (5, 2, 200, 4) and res["dk"].shape == (5, 2, 200, D)
    print(check_forward_backward(w, res))


def test_explicit_scale_and_given_indices(runner):
    w = workloads.make("scale", "fp32", 2, 2, 96, 32, 16, 3, 20, seed=5)
    p, res = run(runner, w, sm_scale=0.37)
    print(check_forward_backward(w, res, sm_scale=0.37))
    # indices as input: hand the library a different, valid selection and compare with the
    # oracle run on the same indices
    idx = res["idx"].copy()
    idx[:, :, 3:, 0] = 0
    idx[:, :, 3:, 1] = 2
    idx[:, :, 3:, 2] = np.arange(3, w.n_blocks)[None, None, :]
    import torch
    p.idx.copy_(torch.from_numpy(idx))
    p.forward(idx_is_input=True)
    p.backward()
    res2 = p.results()
    assert np.array_equal(res2["idx"], idx)
    import oracle
    ref = oracle.forward_backward(w.q, w.k, w.v, w.gate, w.dout, w.block, w.topk, w.window,
                                  sm_scale=0.37, idx=idx)
    for key in ("out", "out_lt", "out_st", "lse", "dq", "dk", "dv", "dgate"):
        assert np.abs(res2[key] - ref[key]).max() <= 1e-4, key


def test_inference_mode_and_select_only(runner):
    w = workloads.config2(B=8)
    p, res = run(runner, w)
    q, _ = run(runner, w, training=False, backward=False)
    r2 = q.results()
    assert np.array_equal(r2["out"], res["out"]) and np.array_equal(r2["idx"], res["idx"])
    q.idx.fill_(-7)
    q.select()
    assert np.array_equal(q.results()["idx"], res["idx"])


@pytest.mark.parametrize("opts", [{}, {"kv_heads": 2}, {"per_query": 1}, {"causal": 0}, {"rope_theta": 10000.0},
                                  {"rope_theta": 500.0, "dtype": "fp32"}])
def test_backward_on_the_forward_s_tile_lists_gives_the_same_bits(runner, opts):
    """reuse_tile_lists = 1: a backward call that follows a training forward on the same workspace
    walks the lists that forward built and, with rotary positions, reads the rotated q and k that
    forward left there; the gradients are those of a backward that builds its own, bit for bit."""
    w = workloads.make("reuse-lists", opts.get("dtype", "bf16"), 3, 4, 900, 64, 32, 5, 70, seed=89, lengths=(200, 900),
                       kv_heads=opts.get("kv_heads", 0))
    w.per_query, w.causal = opts.get("per_query", 0), opts.get("causal", 1)
    w.rope_theta = opts.get("rope_theta", 0.0)
    p = runner.DeviceProblem(w)
    p.forward()
    p.backward(reuse_tile_lists=False)
    own = p.results()
    for t in (p.dq, p.dk, p.dv, p.dgate):
        t.fill_(7.0)
    p.forward()
    p.backward(reuse_tile_lists=True)
    reused = p.results()
    for key in ("dq", "dk", "dv", "dgate"):
        assert np.array_equal(own[key], reused[key]), key
    print(check_forward_backward(w, reused))


def test_host_pipeline_returns_the_device_resident_results(runner):
    """Steps streamed from and to pinned host memory over alternating device slots give, step
    after step, the bits of a device-resident step."""
    import torch
    w = workloads.make("pipe", "bf16", 3, 2, 700, 64, 32, 5, 70, seed=31, lengths=(100, 700))
    p, res = run(runner, w)
    pipe = runner.HostPipeline(w, slots=2)
    h_in = pipe.pinned_inputs()
    outs = [pipe.pinned_outputs() for _ in range(5)]
    for o in outs:
        for t in o.values():
            t.fill_(7.0)
        pipe.submit(h_in, o)
    pipe.drain()
    for o in outs:
        for k in ("out", "dq", "dk", "dv", "dgate"):
            assert np.array_equal(o[k].float().numpy(), res[k]), k


def test_step_replays_from_a_cuda_graph(runner):
    """Selection, forward and backward launch on the caller's stream and allocate nothing, so a
    step can be captured once and replayed; the replays give the bits of the eager step."""
    import torch
    w = workloads.make("graph", "bf16", 2, 2, 600, 64, 32, 4, 96, seed=37, lengths=(200, 600))
    p, res = run(runner, w)
    for name in ("out", "dq", "dk", "dv", "dgate", "idx"):
        getattr(p, name).zero_()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        p.step()                      # warm-up on the capture stream (attributes, tensor maps)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            p.step()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        for name in ("out", "dq", "dk", "dv", "dgate"):
            getattr(p, name).zero_()
        graph.replay()
        got = p.results()
        for k in ("idx", "out", "out_lt", "out_st", "lse", "dq", "dk", "dv", "dgate"):
            assert np.array_equal(got[k], res[k]), k


def test_strided_layout(runner):
    """q-shaped tensors stored [B, L, H, D] (the layout a fused QKV projection produces)."""
    import torch
    from paper_2512_13368_b200 import binding
    w = workloads.make("strided", "bf16", 2, 4, 160, 64, 32, 3, 40, seed=8)
    p = runner.DeviceProblem(w)
    perm = lambda t: t.permute(0, 2, 1, 3).contiguous()          # noqa: E731  memory [B,L,H,D]
    bufs = {k: perm(getattr(p, k)) for k in ("q", "k", "v", "dout")}
    outs = {k: torch.empty_like(bufs["q"]) for k in ("out", "out_lt", "out_st", "dq", "dk", "dv")}
    prm = binding.make_params(w.B, w.H, w.L, w.D, w.block, w.topk, w.window, w.dtype,
                              strides=(w.L * w.H * w.D, w.D, w.H * w.D))
    binding.blossom_attn_fwd(prm, bufs["q"], bufs["k"], bufs["v"], p.gate, None, p.idx, 0, outs["out"],
                             outs["out_lt"], outs["out_st"], p.lse, p.workspace)
    binding.blossom_attn_bwd(prm, bufs["q"], bufs["k"], bufs["v"], p.gate, None, p.idx, outs["out_lt"],
                             outs["out_st"], p.lse, bufs["dout"], outs["dq"], outs["dk"], outs["dv"],
                             p.dgate, p.workspace)
    torch.cuda.synchronize()
    res = {k: v.permute(0, 2, 1, 3).float().cpu().numpy() for k, v in outs.items()}
    res.update(idx=p.idx.cpu().numpy(), lse=p.lse.cpu().numpy(), dgate=p.dgate.cpu().numpy())
    print(check_forward_backward(w, res))


def test_constructed_ties_pick_lower_index(runner):
    """Exact ties in the block scores: identical key blocks give bit-identical scores."""
    rng = np.random.default_rng(3)
    B, H, L, D, block, topk = 1, 2, 128, 32, 16, 3
    w = workloads.make("ties", "bf16", B, H, L, D, block, topk, 8, seed=9)
    blk = workloads.quantize(rng.standard_normal((D,)).astype(np.float32), "bf16")
    w.k[:] = blk[None, None, None, :]          # every key identical -> all block scores tie
    _, res = run(runner, w, backward=False)
    for b in range(L // block):
        exp = list(range(min(b, topk - 1))) + [b]
        exp += [-1] * (topk - len(exp))
        assert list(res["idx"][0, 0, b]) == exp and list(res["idx"][0, 1, b]) == exp
    assert check_indices(w, res["idx"]) == 0


# ------------------------------------------------- full benchmark sizes, every output element
def _whole_batch(runner, w):
    """One step at the full benchmark size, in the launch configuration the benchmark times, and
    every element of every output (indices, out, out_lt, out_st, lse, dq, dk, dv and the gate
    gradient, which is a sum over the whole batch) compared with the oracle run on the whole
    batch (it parallelises over (batch, head) units by itself)."""
    p = runner.DeviceProblem(w)
    p.step()
    from paper_2512_13368_b200 import binding
    assert binding.blossom_device_status(p.workspace) == 0
    res = p.results()
    errs = check_forward_backward(w, res)
    assert "dgate" in errs and "dk" in errs
    return errs, res


def test_config3_full_size(runner):
    errs, _ = _whole_batch(runner, workloads.config3())
    print(errs)


def test_config4_full_size(runner):
    errs, _ = _whole_batch(runner, workloads.config4())
    print(errs)


def test_config5_attention_shape_full_batch(runner):
    errs, _ = _whole_batch(runner, workloads.config5_attention())
    print(errs)


def test_config4_full_size_grouped_heads(runner):
    """The headline shape with its 8 query heads on 2 key/value heads, as the benchmark's
    --kv-heads 2 option times it."""
    w = workloads.config4(kv_heads=2)
    errs, res = _whole_batch(runner, w)
    print(errs)
    assert res["idx"].shape == (w.B, 2, w.n_blocks, w.topk) and res["dk"].shape == w.k.shape


def test_config4_full_size_overlapping_compression(runner):
    """The headline shape with compression blocks of 128 keys at stride 32 behind the selection,
    as the benchmark's --cmp-block 128 --cmp-stride 32 option times it."""
    w = workloads.config4()
    w.cmp_block, w.cmp_stride = 128, 32
    errs, _ = _whole_batch(runner, w)
    print(errs)


def test_config4_full_size_power_law(runner):
    """The headline shape with the paper's short-term mask (window 8, mask block 1), in the launch
    configuration the benchmark's --short-term power-law option times."""
    w = workloads.config4()
    w.stis_mode, w.stis_block, w.window = 1, 1, 8
    errs, _ = _whole_batch(runner, w)
    print(errs)


def test_config4_full_size_paper_options_together(runner):
    """The headline shape with the paper's three options at once (8 heads on 2 key/value heads,
    overlapping compression blocks 128 / 32 behind the 64-position selection blocks, power-law
    mask with window 8 and mask block 1), as the benchmark's --paper-options times it."""
    w = workloads.config4(kv_heads=2)
    w.cmp_block, w.cmp_stride = 128, 32
    w.stis_mode, w.stis_block, w.window = 1, 1, 8
    errs, _ = _whole_batch(runner, w)
    print(errs)


def test_config4_full_size_paper_options_with_the_selection_per_query_position(runner):
    """The headline shape with all of the paper's options and its per-position selection, as the
    benchmark's --paper-options --per-query times it."""
    w = workloads.config4(kv_heads=2)
    w.cmp_block, w.cmp_stride, w.per_query = 128, 32, 1
    w.stis_mode, w.stis_block, w.window = 1, 1, 8
    errs, res = _whole_batch(runner, w)
    print(errs)
    assert res["idx"].shape == (w.B, 2, w.L, w.topk)


def test_config2_full_size(runner):
    w = workloads.config2()
    errs, res = _whole_batch(runner, w)
    print(errs)
    # structure of every index row, zero padding
    idx = res["idx"]
    M = w.n_blocks
    own = np.arange(M)[None, None, :]
    last = np.where(idx >= 0, idx, -1).max(-1)
    pad0 = w.L - w.seq_lens
    live_block = (np.minimum((np.arange(M) + 1) * w.block, w.L)[None, :] > pad0[:, None])
    assert np.all(np.where(live_block[:, None, :], last == own, last == -1))
    for n in range(w.B):
        for key in ("out", "out_lt", "out_st", "dq", "dk", "dv"):
            assert np.all(res[key][n, :, :pad0[n]] == 0.0)


def _fast_and_exact_selection(p):
    """The indices of the two-stage selection and of the double-precision-only selection."""
    import torch
    from paper_2512_13368_b200 import binding
    binding.blossom_debug_switch(binding.SWITCH_EXACT_SELECT, 0)
    try:
        p.select()
        torch.cuda.synchronize()
        fast = p.idx.cpu().numpy().copy()
        binding.blossom_debug_switch(binding.SWITCH_EXACT_SELECT, 1)
        p.idx.fill_(-7)
        p.select()
        torch.cuda.synchronize()
        exact = p.idx.cpu().numpy().copy()
    finally:
        binding.blossom_debug_switch(binding.SWITCH_EXACT_SELECT, -1)
    return fast, exact


def test_certified_selection_equals_double_precision_selection(runner):
    """The two-stage selection (fp32 scores with an error bound, fp64 only for the uncertain query
    blocks) must return exactly what scoring every query block in fp64 returns."""
    import torch
    overlap4 = workloads.config4(B=1)
    overlap4.cmp_block, overlap4.cmp_stride = 128, 32          # 125 compression blocks: two chunks
    overlap2 = workloads.config2(B=16)
    overlap2.cmp_block, overlap2.cmp_stride = 32, 16           # the paper's default sizes, padded rows
    small_stride = workloads.make("small-stride", "bf16", 1, 2, 2048, 32, 16, 6, 16, seed=9)
    small_stride.cmp_block, small_stride.cmp_stride = 32, 8    # 253 compression blocks: four chunks
    gqa_overlap = workloads.config2(B=16, kv_heads=1)
    gqa_overlap.cmp_block, gqa_overlap.cmp_stride = 32, 16     # grouped heads through overlapping blocks
    gqa_overlap4 = workloads.config4(B=1, kv_heads=2)
    gqa_overlap4.cmp_block, gqa_overlap4.cmp_stride = 128, 32
    for w in (workloads.config4(B=1), workloads.config2(B=16), workloads.config3(B=1), gqa_overlap, gqa_overlap4,
              workloads.config4(B=1, kv_heads=2), workloads.config2(B=16, kv_heads=1),
              workloads.config3(B=1, kv_heads=1),
              workloads.make("many-blocks", "bf16", 1, 2, 2048, 32, 16, 6, 16, seed=9),
              overlap4, overlap2, small_stride):
        p = runner.DeviceProblem(w)
        fast, exact = _fast_and_exact_selection(p)
        assert np.array_equal(fast, exact), w.name
        check_indices(w, fast)


def test_certified_selection_on_random_small_block_shapes(runner):
    """Short sequences of 16- and 32-position blocks take the first-stage kernel that packs
    several query blocks into a CTA: over random shapes, lengths, scales and exact ties (identical
    keys) its choice must be the double-precision one, bit for bit."""
    import torch
    rng = np.random.default_rng(123)
    for it in range(48):
        Bk = int(rng.choice([16, 32]))
        M = int(rng.integers(1, 65))
        L = int(rng.integers((M - 1) * Bk + 1, M * Bk + 1))
        D = int(rng.choice([32, 64]))
        H, B = int(rng.choice([1, 2, 3])), int(rng.integers(1, 5))
        topk, dtype = int(rng.integers(1, 12)), str(rng.choice(["bf16", "fp32"]))
        std = float(rng.choice([0.05, 0.5, 1.0, 3.0]))
        lens = None if rng.random() < 0.4 else (1, L)
        w = workloads.make("rand-small", dtype, B, H, L, D, Bk, topk, 16, seed=1000 + it, std=std, lengths=lens)
        if it % 7 == 0:
            w.k[:] = w.k[:, :, :1, :]      # every key equal: every score ties
        p = runner.DeviceProblem(w)
        fast, exact = _fast_and_exact_selection(p)
        assert np.array_equal(fast, exact), (it, L, Bk, D, H, B, topk, dtype, std)


def _random_option_workload(rng, it):
    """A small bf16 / fp32 problem with a random legal combination of the options."""
    Bk = int(rng.choice([16, 32, 64]))
    D = int(rng.choice([32, 64]))
    Hkv = int(rng.choice([1, 2]))
    H = Hkv * int(rng.choice([1, 2]))
    L = int(rng.integers(Bk + 1, 700))
    topk, window = int(rng.integers(1, 7)), int(rng.integers(1, 90))
    dtype = "bf16" if rng.random() < 0.8 else "fp32"
    lens = None if rng.random() < 0.4 else (0, L)
    power_law = rng.random() < 0.4
    w = workloads.make(f"rand-options-{it}", dtype, 3, H, L, D, Bk, topk, window, seed=2000 + it, lengths=lens,
                       kv_heads=Hkv if Hkv != H else 0, stis_mode=1 if power_law else 0,
                       stis_block=int(rng.choice([1, 2, 4])) if power_law else 1)
    w.causal = 0 if rng.random() < 0.3 else 1
    if w.causal:
        if rng.random() < 0.4:
            w.per_query = 1
        if rng.random() < 0.4:
            s = int(rng.choice([x for x in (4, 8, 16, 32, 64) if Bk % x == 0]))
            w.cmp_block, w.cmp_stride = s * int(rng.choice([1, 2, 4])), s
            if w.per_query and ((L - w.cmp_block) // s + 1 > 128 or -(-L // Bk) > 128):
                w.cmp_block = w.cmp_stride = 0
    if rng.random() < 0.3:
        w.gate_mode = 1
        w.gate = (0.3 * rng.standard_normal((H, 2 * D + 1))).astype(np.float32)
    if rng.random() < 0.3:
        w.rope_theta = 10000.0
    if rng.random() < 0.3:
        w.phi_logits = rng.standard_normal(w.cmp_block or Bk).astype(np.float32)
    return w


def test_random_combinations_of_the_options(runner):
    """Forty seeded problems with random shapes, lengths and legal combinations of the options
    (power-law mask, compression blocks, grouped heads, per-position selection, pooled summaries,
    input-dependent gate, no causal mask, rotary positions), each against the oracle."""
    rng = np.random.default_rng(2024)
    for it in range(40):
        w = _random_option_workload(rng, it)
        _, res = run(runner, w)
        try:
            check_forward_backward(w, res)
        except AssertionError as e:
            raise AssertionError(f"case {it}: {w}: {e}") from e


@pytest.mark.parametrize("opts", [{}, {"causal": 0}, {"per_query": 1}, {"gate_mode": 1}, {"power_law": True, "kv_heads": 2},
                                  {"full": True}, {"full": True, "causal": 0}, {"full": True, "kv_heads": 2}])
def test_repeated_steps_give_the_same_bits(runner, opts):
    """Nothing in the path is allowed to depend on the order in which warps or CTAs happen to run
    (no atomics on results, fixed reduction orders, every hand-off behind a barrier): repeated
    steps on the same inputs, with the outputs poisoned in between, must give identical bits
    (thirty steps of a mid-size problem, twelve of the headline shape)."""
    import torch
    if opts.get("full"):
        w, reps = workloads.config4(kv_heads=opts.get("kv_heads", 0)), 12
    else:
        w, reps = workloads.make("repeat", "bf16", 4, 4, 2048, 64, 64, 8, 200, seed=97, lengths=(700, 2048),
                                 kv_heads=opts.get("kv_heads", 0), stis_mode=1 if opts.get("power_law") else 0), 30
    w.causal, w.per_query, w.gate_mode = opts.get("causal", 1), opts.get("per_query", 0), opts.get("gate_mode", 0)
    if w.gate_mode:
        w.gate = (0.3 * np.random.default_rng(8).standard_normal((w.H, 2 * w.D + 1))).astype(np.float32)
    p = runner.DeviceProblem(w)
    p.step()
    keys = ("idx", "out", "out_lt", "out_st", "lse", "dq", "dk", "dv", "dgate")
    first = {k: getattr(p, k).clone() for k in keys}
    for it in range(reps):
        for k in keys:
            getattr(p, k).view(torch.uint8).fill_(0xFF)
        p.step()
        for k in keys:
            assert torch.equal(first[k].view(torch.uint8), getattr(p, k).view(torch.uint8)), (it, k)
    if opts.get("full"):
        # the forward alone, many more times: a missing barrier between its two phases once showed
        # as a few wrong long-term rows in one of ~25 (non-causal) to ~150 (causal) launches
        fkeys = ("out", "out_lt", "out_st", "lse")
        for it in range(400):
            p.forward(True)
            for k in fkeys:
                assert torch.equal(first[k].view(torch.uint8), getattr(p, k).view(torch.uint8)), (it, k)
    from paper_2512_13368_b200 import binding
    assert binding.blossom_device_status(p.workspace) == 0
    if not opts.get("full"):
        print(check_forward_backward(w, p.results()))


@pytest.mark.parametrize("opts", [{}, {"kv_heads": 2, "power_law": True}, {"per_query": 1}, {"gate_mode": 1}])
def test_chained_and_serial_launches_give_the_same_bits(runner, opts):
    """By default a kernel of a call may become resident while the last CTAs of the kernel before it
    still run, and waits for that kernel's completion before it touches global memory; with the
    debugging switch every launch is fully serialised.  Same bits either way, steps alternating."""
    import torch
    from paper_2512_13368_b200 import binding
    w = workloads.make("chained", "bf16", 4, 4, 1500, 64, 32, 6, 100, seed=53, lengths=(300, 1500),
                       kv_heads=opts.get("kv_heads", 0), stis_mode=1 if opts.get("power_law") else 0)
    w.per_query, w.gate_mode = opts.get("per_query", 0), opts.get("gate_mode", 0)
    if w.gate_mode:
        w.gate = (0.3 * np.random.default_rng(9).standard_normal((w.H, 2 * w.D + 1))).astype(np.float32)
    p = runner.DeviceProblem(w)
    keys = ("idx", "out", "out_lt", "out_st", "lse", "dq", "dk", "dv", "dgate")
    try:
        binding.blossom_debug_switch(binding.SWITCH_SERIAL_LAUNCH, 1)
        p.step()
        first = {k: getattr(p, k).clone() for k in keys}
        for it in range(12):
            binding.blossom_debug_switch(binding.SWITCH_SERIAL_LAUNCH, it % 2)
            for k in keys:
                getattr(p, k).view(torch.uint8).fill_(0xFF)
            for _ in range(3):
                p.step()
            for k in keys:
                assert torch.equal(first[k].view(torch.uint8), getattr(p, k).view(torch.uint8)), (it, k)
    finally:
        binding.blossom_debug_switch(binding.SWITCH_SERIAL_LAUNCH, -1)
    assert binding.blossom_device_status(p.workspace) == 0
    print(check_forward_backward(w, p.results()))


def test_profile_of_every_nth_launch(runner):
    """blossom_profile_every(n): only every n-th launch of each kernel is bracketed by events."""
    from paper_2512_13368_b200 import binding
    w = workloads.make("sampled", "bf16", 2, 2, 512, 64, 64, 4, 100, seed=5)
    p = runner.DeviceProblem(w)
    p.step()
    counts = {}
    for every in (1, 3):
        binding.blossom_profile_every(every)
        binding.blossom_profile_start(256)
        for _ in range(6):
            p.step()
        rec = binding.blossom_profile_stop(256)
        counts[every] = {}
        for name, ms in rec:
            assert ms > 0.0
            counts[every][name] = counts[every].get(name, 0) + 1
    binding.blossom_profile_every(1)
    assert counts[1]["fwd_tc"] == 6 and counts[3]["fwd_tc"] == 2
    assert set(counts[1]) == set(counts[3])
    assert all(counts[3][k] * 3 == counts[1][k] for k in counts[1])
    with pytest.raises(binding.BlossomError):
        binding.blossom_profile_every(0)


# ------------------------------------------- what stands in for a memory checker on this path
def _guarded(shape, dtype, fill, device, pad=4096):
    """A tensor carved out of a larger allocation with `pad` guard elements before and after it."""
    import torch
    n = int(np.prod(shape))
    raw = torch.full((n + 2 * pad,), fill, dtype=dtype, device=device)
    return raw, raw[pad:pad + n].view(shape)


@pytest.mark.parametrize("L,D,block,topk,window,lens,kv_heads", [
    (200, 32, 16, 4, 32, [200, 77, 5], 0),      # ragged last block and last tile, padded batch entries
    (330, 64, 32, 5, 70, [330, 129], 0),        # L not a multiple of 64: the bulk stores are clipped at L
    (257, 64, 64, 3, 300, None, 2),             # one row past a tile border, grouped heads
])
def test_no_write_outside_any_output(runner, L, D, block, topk, window, lens, kv_heads):
    """Every output (out, out_lt, out_st, lse, dq, dk, dv, dgate, block_idx) sits between guard
    regions that must come back untouched: the tensor-core kernels write their results with bulk
    tensor stores that rely on the hardware clipping rows past L, and nothing else would notice a
    store that strays."""
    import torch
    from paper_2512_13368_b200 import binding
    B = len(lens) if lens else 2
    H = 4
    w = workloads.make("guards", "bf16", B, H, L, D, block, topk, window, seed=43, kv_heads=kv_heads)
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    p = runner.DeviceProblem(w)
    dev = p.q.device
    hkv = kv_heads or H
    bf, f32, i32 = torch.bfloat16, torch.float32, torch.int32
    specs = {"out": ((B, H, L, D), bf), "out_lt": ((B, H, L, D), bf), "out_st": ((B, H, L, D), bf),
             "dq": ((B, H, L, D), bf), "dk": ((B, hkv, L, D), bf), "dv": ((B, hkv, L, D), bf),
             "lse": ((2, B, H, L), f32), "dgate": ((H, 2), f32), "idx": ((B, hkv, w.n_blocks, topk), i32)}
    raws = {}
    for name, (shape, dt) in specs.items():
        fill = -7 if dt == i32 else 123.0
        raws[name], view = _guarded(shape, dt, fill, dev)
        setattr(p, name, view)
    p.step()
    assert binding.blossom_device_status(p.workspace) == 0
    res = p.results()
    for name, (shape, dt) in specs.items():
        raw, n, fill = raws[name], int(np.prod(shape)), (-7 if dt == i32 else 123.0)
        assert bool((raw[:4096] == fill).all()) and bool((raw[4096 + n:] == fill).all()), name
    print(check_forward_backward(w, res))


@pytest.mark.parametrize("cfg", ["cfg2", "cfg3", "edge"])
def test_tensor_core_path_against_the_cuda_core_path(runner, cfg):
    """A second opinion on the tensor-core kernels: the same bf16 problem through the fp32
    CUDA-core kernels (debugging switch), which share none of their code.  Both round their
    outputs to bf16, so they agree to a few bf16 units in the last place of the largest value."""
    from paper_2512_13368_b200 import binding
    if cfg == "cfg2":
        w = workloads.config2(B=16)
    elif cfg == "cfg3":
        w = workloads.config3(B=1)
    else:
        w = workloads.make("edge-simt", "bf16", 2, 3, 700, 32, 16, 9, 48, seed=47, lengths=(100, 700))
    _, tc = run(runner, w)
    binding.blossom_debug_switch(binding.SWITCH_FORCE_SIMT, 1)
    try:
        _, simt = run(runner, w)
    finally:
        binding.blossom_debug_switch(binding.SWITCH_FORCE_SIMT, -1)
    assert np.array_equal(tc["idx"], simt["idx"])
    for key in ("out", "out_lt", "out_st", "lse", "dq", "dk", "dv", "dgate"):
        ref = np.abs(simt[key]).max()
        err = np.abs(tc[key] - simt[key]).max()
        assert err <= 2e-2 * max(ref, 1e-3), (key, err, ref)
    check_forward_backward(w, simt)      # and the CUDA-core path against the oracle


def test_a_wait_that_cannot_complete_is_reported_and_the_context_stays_usable(runner):
    """The timeout branch of the bounded device-side waits, in the allowed form: a diagnostic
    kernel waits on a barrier nobody arrives at; the wait gives up after its limit, the kernel ends
    normally, frees its tensor memory and leaves BLOSSOM_ERR_TIMEOUT, the site of the wait and the
    CTA in the status words.  A normal step afterwards must still be right."""
    import torch
    from paper_2512_13368_b200 import binding
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda:0")
    binding.blossom_selftest_wait_timeout(ws)
    assert binding.blossom_device_status(ws) == binding.BLOSSOM_ERR_TIMEOUT
    words = ws[:16].cpu().numpy().view(np.int32)
    assert words[0] == binding.BLOSSOM_ERR_TIMEOUT and 900 <= words[1] < 904 and words[2] == 0
    w = workloads.make("after-timeout", "bf16", 2, 2, 300, 64, 32, 3, 50, seed=53)
    _, res = run(runner, w)                    # tensor memory was freed, barriers work, results are right
    print(check_forward_backward(w, res))


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("L,D,H,Hkv,block,topk,window,lens,power_law", [
    (64, 32, 2, 2, 8, 2, 16, None, False),
    (200, 32, 2, 2, 16, 4, 32, [200, 5, 77, 0], False),      # padded, ragged last block
    (300, 64, 4, 2, 32, 4, 40, [300, 131], False),           # grouped heads share a per-position selection
    (257, 64, 2, 2, 64, 3, 8, None, True),                   # with the power-law short-term mask
    (1024, 64, 2, 2, 64, 8, 64, [1024, 700], False),
    (300, 64, 4, 2, 32, 4, 40, [300, 131], "cmp64/16"),      # through overlapping compression blocks
    (1000, 32, 2, 2, 16, 5, 30, [1000, 404], "cmp32/8"),     # 122 compression blocks: two chunks
])
def test_selection_per_query_position(runner, dtype, L, D, H, Hkv, block, topk, window, lens, power_law):
    """select_mode 1 (Eq. 13 as the paper prints it: every query position keeps its own top-k
    blocks): indices, forward and backward against the oracle."""
    B = len(lens) if lens else 2
    w = workloads.make("per-query", dtype, B, H, L, D, block, topk, window, seed=59, kv_heads=Hkv if Hkv != H else 0,
                       stis_mode=1 if power_law is True else 0)
    w.per_query = 1
    if isinstance(power_law, str):
        w.cmp_block, w.cmp_stride = (int(x) for x in power_law[3:].split("/"))
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    _, res = run(runner, w)
    assert res["idx"].shape == (B, Hkv, L, topk)
    print(check_forward_backward(w, res))


@pytest.mark.parametrize("block,power_law", [(16, False), (32, True), (64, False)])
def test_selection_per_query_position_runs_on_the_tensor_core_kernels(runner, block, power_law):
    """bf16 shapes of up to 4096 positions keep the tensor-core kernels with select_mode 1 (their
    tile lists are the union of a query block's rows, every row masks with its own selection):
    the launch record shows those kernels, and the results agree with the oracle and with the
    CUDA-core path."""
    from paper_2512_13368_b200 import binding
    w = workloads.make("per-query-tc", "bf16", 3, 4, 1000, 64, block, 5, 70, seed=79, kv_heads=2, lengths=(300, 1000),
                       stis_mode=1 if power_law else 0, stis_block=2 if power_law else 1)
    w.per_query = 1
    binding.blossom_profile_start(64)
    _, tc = run(runner, w)
    names = {name for name, _ in binding.blossom_profile_stop(64)}
    assert {"fwd_tc", "bwd_dq_tc", "bwd_dkdv_tc"} <= names and not any("simt" in x for x in names), names
    assert tc["idx"].shape == (w.B, 2, w.L, w.topk)
    print(check_forward_backward(w, tc))
    binding.blossom_debug_switch(binding.SWITCH_FORCE_SIMT, 1)
    try:
        _, simt = run(runner, w)
    finally:
        binding.blossom_debug_switch(binding.SWITCH_FORCE_SIMT, -1)
    assert np.array_equal(tc["idx"], simt["idx"])
    for key in ("out", "out_lt", "out_st", "lse", "dq", "dk", "dv", "dgate"):
        ref = np.abs(simt[key]).max()
        err = np.abs(tc[key] - simt[key]).max()
        assert err <= 2e-2 * max(ref, 1e-3), (key, err, ref)


def test_config4_full_size_selection_per_query_position(runner):
    """The headline shape with a selection per query position, as the benchmark's --per-query
    option times it."""
    w = workloads.config4()
    w.per_query = 1
    errs, res = _whole_batch(runner, w)
    print(errs)
    assert res["idx"].shape == (w.B, w.H, w.L, w.topk)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("L,D,H,Hkv,block,topk,cmp,lens,per_query", [
    (200, 32, 2, 2, 16, 4, None, [200, 5, 77], False),
    (512, 64, 4, 2, 32, 4, (64, 16), [512, 200], False),     # overlapping blocks, grouped heads
    (1024, 64, 2, 2, 64, 6, None, None, False),
    (192, 32, 2, 2, 16, 3, None, [192, 40], True),           # with a selection per query position
])
def test_learnable_block_summary(runner, dtype, L, D, H, Hkv, block, topk, cmp, lens, per_query):
    """Eq. 9's learnable summary (softmax pooling over a block's positions, logits given by the
    caller) behind the selection: indices bit-checked against the oracle, attention on them."""
    B = len(lens) if lens else 2
    w = workloads.make("phi", dtype, B, H, L, D, block, topk, 24, seed=61, kv_heads=Hkv if Hkv != H else 0)
    if cmp:
        w.cmp_block, w.cmp_stride = cmp
    w.per_query = int(per_query)
    w.phi_logits = np.random.default_rng(3).standard_normal(cmp[0] if cmp else block).astype(np.float32)
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    _, res = run(runner, w)
    print(check_forward_backward(w, res))
    # the logits matter: the mean selects something else somewhere
    w0 = workloads.make("phi", dtype, B, H, L, D, block, topk, 24, seed=61, kv_heads=Hkv if Hkv != H else 0)
    if cmp:
        w0.cmp_block, w0.cmp_stride = cmp
    w0.per_query, w0.seq_lens = w.per_query, w.seq_lens
    _, res0 = run(runner, w0, backward=False)
    assert not np.array_equal(res0["idx"], res["idx"])


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("L,D,H,Hkv,block,topk,window,lens,per_query", [
    (64, 32, 2, 2, 8, 2, 16, None, False),
    (200, 32, 2, 2, 16, 4, 32, [200, 5, 77, 0], False),
    (300, 64, 4, 2, 32, 4, 40, [300, 131], False),            # grouped heads
    (257, 64, 2, 2, 64, 3, 8, None, True),                    # with a selection per query position
])
def test_input_dependent_gate(runner, dtype, L, D, H, Hkv, block, topk, window, lens, per_query):
    """gate_mode 1 (Eq. 18: alpha = sigmoid(F_o([O_lt; O_st])) per query row with a one-layer F_o,
    Eq. 19): forward, the gradients of q, k, v and of F_o's parameters against the oracle."""
    B = len(lens) if lens else 2
    w = workloads.make("gate-mlp", dtype, B, H, L, D, block, topk, window, seed=67, kv_heads=Hkv if Hkv != H else 0)
    w.gate_mode, w.per_query = 1, int(per_query)
    w.gate = (0.3 * np.random.default_rng(5).standard_normal((H, 2 * D + 1))).astype(np.float32)
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    _, res = run(runner, w)
    assert res["dgate"].shape == (H, 2 * D + 1)
    print(check_forward_backward(w, res))


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("L,D,H,Hkv,block,topk,window,lens,power_law", [
    (64, 32, 2, 2, 8, 3, 5, None, False),
    (200, 32, 2, 2, 16, 4, 9, [200, 5, 77, 0], False),       # padded, ragged last block
    (300, 64, 4, 2, 32, 4, 17, [300, 131], True),            # grouped heads, symmetric power-law mask
    (512, 64, 2, 2, 64, 8, 600, None, False),                # everything visible: dense bidirectional attention
])
def test_without_the_causal_mask(runner, dtype, L, D, H, Hkv, block, topk, window, lens, power_law):
    """causal = 0 (the bidirectional encoders of the paper's transfer experiment): selection among
    all other live blocks, attention over whole selected blocks, symmetric Eq. 15."""
    B = len(lens) if lens else 2
    w = workloads.make("non-causal", dtype, B, H, L, D, block, topk, window, seed=73, kv_heads=Hkv if Hkv != H else 0,
                       stis_mode=1 if power_law else 0, stis_block=2 if power_law else 1)
    w.causal = 0
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    _, res = run(runner, w)
    print(check_forward_backward(w, res))


@pytest.mark.parametrize("block,power_law", [(16, False), (32, True), (64, False)])
def test_without_the_causal_mask_runs_on_the_tensor_core_kernels(runner, block, power_law):
    """bf16 shapes keep the tensor-core kernels with causal = 0 (tile lists over both sides of the
    diagonal, whole selected blocks, the symmetric short-term mask): the launch record shows those
    kernels, and the results agree with the oracle and with the CUDA-core path."""
    from paper_2512_13368_b200 import binding
    w = workloads.make("non-causal-tc", "bf16", 3, 4, 1000, 64, block, 5, 70, seed=83, kv_heads=2, lengths=(300, 1000),
                       stis_mode=1 if power_law else 0, stis_block=2 if power_law else 1)
    w.causal = 0
    binding.blossom_profile_start(64)
    _, tc = run(runner, w)
    names = {name for name, _ in binding.blossom_profile_stop(64)}
    assert {"fwd_tc", "bwd_dq_tc", "bwd_dkdv_tc"} <= names and not any("simt" in x for x in names), names
    print(check_forward_backward(w, tc))
    binding.blossom_debug_switch(binding.SWITCH_FORCE_SIMT, 1)
    try:
        _, simt = run(runner, w)
    finally:
        binding.blossom_debug_switch(binding.SWITCH_FORCE_SIMT, -1)
    assert np.array_equal(tc["idx"], simt["idx"])
    for key in ("out", "out_lt", "out_st", "lse", "dq", "dk", "dv", "dgate"):
        ref = np.abs(simt[key]).max()
        err = np.abs(tc[key] - simt[key]).max()
        assert err <= 2e-2 * max(ref, 1e-3), (key, err, ref)


def test_config4_full_size_without_the_causal_mask(runner):
    """The headline shape without the causal mask, as the benchmark's --non-causal option times it."""
    w = workloads.config4()
    w.causal = 0
    errs, _ = _whole_batch(runner, w)
    print(errs)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("L,D,H,Hkv,block,topk,window,lens", [
    (64, 32, 2, 2, 8, 2, 16, None),
    (200, 32, 2, 2, 16, 4, 32, [200, 5, 77, 0]),
    (700, 64, 4, 2, 32, 5, 70, [700, 129]),              # tensor-core kernels (bf16) on the rotated copies
    (1024, 64, 2, 2, 64, 8, 256, None),
])
def test_rotary_positions_inside_the_library(runner, dtype, L, D, H, Hkv, block, topk, window, lens):
    """rope_theta > 0: q and k are rotated by position inside the library before the selection and
    both branches, and the backward returns gradients with respect to the unrotated q and k."""
    B = len(lens) if lens else 2
    w = workloads.make("rope", dtype, B, H, L, D, block, topk, window, seed=79, kv_heads=Hkv if Hkv != H else 0)
    w.rope_theta = 10000.0
    if lens is not None:
        w.seq_lens = np.asarray(lens, dtype=np.int32)
    p, res = run(runner, w)
    print(check_forward_backward(w, res))
    # the inputs are left as they were (the rotated copies live in the workspace)
    assert np.array_equal(p.q.float().cpu().numpy(), w.q) and np.array_equal(p.k.float().cpu().numpy(), w.k)
