"""blossom_select_blocks_static: the selection entry point for callers that cannot allocate
device memory (no workspace argument; its scratch is a fixed array inside the library).

Collected last on purpose (file name), so a run that stops at the first failure has already run
every other test.  The GPU test calls the entry point through the C ABI several times in a row,
on different problems, and wants exactly the indices the workspace-based entry point returns (the
later calls run on scratch that still holds an earlier call's contents) and the indices the
CPU oracle selects.
"""
import numpy as np
import pytest

from paper_2512_13368_b200 import binding, workloads


def test_capacity_is_checked_on_the_host_before_any_launch():
    binding.load()
    A = 1 << 20  # never dereferenced: the size check comes first
    ok_shape = binding.make_params(16, 8, 4096, 64, 64, 16, 256, "bf16")       # exactly at the limit
    too_many_blocks = binding.make_params(129, 1, 4096, 64, 64, 16, 256, "bf16")
    too_many_means = binding.make_params(16, 8, 8192, 64, 64, 16, 256, "bf16")
    for prm in (too_many_blocks, too_many_means):
        rc = binding.blossom_select_blocks_static(prm, A, A, None, A, stream=0, check=False)
        assert rc == binding.BLOSSOM_ERR_TOO_LARGE
        assert "capacity" in binding.blossom_status_string(rc)
    # argument checks are those of the workspace-based call
    assert binding.blossom_select_blocks_static(ok_shape, None, A, None, A, stream=0, check=False) \
        == binding.BLOSSOM_ERR_INVALID_ARG
    assert binding.blossom_select_blocks_static(ok_shape, A + 2, A, None, A, stream=0, check=False) \
        == binding.BLOSSOM_ERR_INVALID_ARG


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    import torch
    assert torch.cuda.is_available()
    from paper_2512_13368_b200 import runner
    from parity_util import check_indices
    cases = [workloads.config3(B=4),        # first call: L1024, 32 blocks, no padding
             workloads.config2(B=32),       # second call: smaller, left-padded, stale scratch
             workloads.config2(B=24, kv_heads=1),   # grouped heads: scratch indexed per key/value head
             workloads.make("static-gqa", "bf16", 2, 8, 1024, 64, 64, 5, 64, seed=41, kv_heads=2)]
    for w in cases:
        p = runner.DeviceProblem(w)
        p.select()                                           # existing entry point
        torch.cuda.synchronize()
        want = p.idx.cpu().numpy().copy()
        got_t = torch.full_like(p.idx, -7)
        binding.blossom_select_blocks_static(p.params, p.q, p.k, p.seq_lens, got_t)
        torch.cuda.synchronize()
        got = got_t.cpu().numpy()
        assert np.array_equal(got, want), w.name             # integer output: bit-exact
        check_indices(w, got)                                # and the oracle's choice (Eq. 13)
    # and once more on the first problem, now after the smaller one
    w = cases[0]
    p = runner.DeviceProblem(w)
    p.select()
    got_t = torch.full_like(p.idx, -7)
    binding.blossom_select_blocks_static(p.params, p.q, p.k, p.seq_lens, got_t)
    torch.cuda.synchronize()
    assert np.array_equal(got_t.cpu().numpy(), p.idx.cpu().numpy())
