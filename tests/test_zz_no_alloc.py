"""The allocation-free rollout entry point (d2c_op_rollout_static) against d2c_op_rollout.

This file sorts last on purpose: a run that stops at the first failure has then already run every
other test.  The entry point serves callers that cannot obtain device memory when they call (all HBM
already committed to an arena, or a stream on which cudaMalloc's implicit synchronisation is not
acceptable); its scratch is a fixed array inside the library, so two calls in a row reuse the same
memory and the second must not be disturbed by what the first left there.
"""
import numpy as np
import pytest
import torch

from paper_2509_23094_b200 import binding

pytestmark = pytest.mark.gpu


def _case(seed, N, B, L):
    rng = np.random.default_rng(seed)
    nbs = [int(rng.integers(1, L + 1)) for _ in range(B)]
    if B > 2:
        nbs[1] = 0                                                   # a sequence with nothing selected keeps its scores
    row_off = np.concatenate([[0], np.cumsum(nbs)]).astype(np.int32)
    rows = int(row_off[-1])
    sel = np.concatenate([np.sort(rng.choice(L, nb, replace=False)) for nb in nbs]).astype(np.int32)
    abar = rng.random((N, rows, L)).astype(np.float32) ** 3
    abar /= abar.sum(axis=2, keepdims=True)
    return (torch.from_numpy(abar).cuda(), torch.from_numpy(np.concatenate([sel, [0]]).astype(np.int32)).cuda(),
            torch.from_numpy(row_off).cuda())


def test_two_calls_in_a_row_match_the_scratch_taking_entry_point():
    # first a large case that fills most of the built-in scratch, then a small one that reuses a corner of it
    for seed, (N, B, L) in enumerate([(3, 4, 4000), (2, 3, 257)]):
        abar, sel, row_off = _case(seed, N, B, L)
        start = torch.full((B, L), 5.0, dtype=torch.float32, device="cuda")
        want = binding.d2c_op_rollout(abar, sel, row_off, B, L, c=start.clone())
        got = binding.d2c_op_rollout_static(abar, sel, row_off, B, L, c=start.clone())
        torch.cuda.synchronize()
        np.testing.assert_allclose(got.cpu().numpy(), want.cpu().numpy(), rtol=1e-4, atol=1e-5)
        assert torch.all(got[1] == 5.0) if B > 2 else True


def test_sizes_beyond_the_built_in_scratch_are_rejected():
    abar, sel, row_off = _case(9, 1, 1, 64)
    with pytest.raises(binding.D2cError) as e:
        binding.d2c_op_rollout_static(abar, sel, row_off, 3, 8192)     # 24576 positions > 16384
    assert e.value.code == binding.D2C_ECAPACITY and "16384" in str(e.value)
