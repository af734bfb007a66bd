"""The allocation-free variant of the calibration statistic, perq_block_l1_stats_static.

Some users of the library cannot hand it a workspace: a plugin that is only given its input
and output tensors, or a serving loop whose memory pool is fully handed out and whose
allocator must not be called (it could synchronise the device).  For them the library keeps
the per-CTA partial sums in a fixed array of its own.  These tests call that entry point
through the C ABI and hold it to the outputs of the ordinary entry point, twice in a row on
different inputs (the array keeps the previous call's contents, which must not leak).

This file is named so that pytest collects it last.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2601_22347_b200 import inputs


@pytest.fixture(scope="module")
def B():
    from paper_2601_22347_b200 import binding, build
    build.build()
    binding.load()
    return binding


def to_dev(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).cuda().view(torch.bfloat16)


@pytest.mark.gpu
def test_static_scratch_matches_workspace_entry_point_on_two_calls_in_a_row(B):
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    # second call: fewer rows and channels than the first, so stale partial sums of the first
    # call are still in the array beyond what the second one writes
    cases = [(900, 8192, 32, True, 501), (37, 2048, 16, False, 502)]
    for T, d, b, with_perm, seed in cases:
        bits, _ = inputs.swiglu_outliers(T, d, 16, 30.0, seed=seed)
        x = to_dev(bits)
        perm = torch.from_numpy(inputs.random_perm(d, seed + 1)).cuda() if with_perm else None
        ref = B.perq_block_l1_stats(x, perm, b)
        chan = torch.full((d,), -1.0, dtype=torch.float32, device="cuda")
        block = torch.full((d // b,), -1.0, dtype=torch.float32, device="cuda")
        token = torch.full((T,), -1.0, dtype=torch.float32, device="cuda")
        B.perq_block_l1_stats_static(x, perm, b, chan, block, token)
        torch.cuda.synchronize()
        for got, want in zip((chan, block, token), ref):
            # same tolerance as the statistic's parity test; in fact the two are bit-identical
            assert np.allclose(got.cpu().numpy(), want.cpu().numpy(), rtol=1e-5, atol=0)
            assert torch.equal(got, want)
        # only one output requested: the others are left alone
        only = torch.empty(T, dtype=torch.float32, device="cuda")
        B.perq_block_l1_stats_static(x, perm, b, None, None, only)
        torch.cuda.synchronize()
        assert torch.equal(only, ref[2])


def test_static_scratch_rejects_shapes_beyond_its_array_before_touching_cuda(B):
    lib = B.load()
    p = C.c_void_p(0x1000)
    # 148 CTAs x (32768 + 4096) floats does not fit 148 x 16384
    assert lib.perq_block_l1_stats_static(p, None, 4096, 32768, 8, p, p, p, None) == 9
    assert lib.perq_block_l1_stats_static(p, None, 148 * 28, 16384, 16384, p, p, p, None) == 9   # 148 x 16385
    # shape errors are reported as for the ordinary entry point
    assert lib.perq_block_l1_stats_static(p, None, 16, 4100, 32, p, p, p, None) == 2
    assert lib.perq_block_l1_stats_static(p, None, 16, 4096, 24, p, p, p, None) == 3
    # nothing requested: nothing to do
    assert lib.perq_block_l1_stats_static(p, None, 16, 4096, 32, None, None, None, None) == 0
