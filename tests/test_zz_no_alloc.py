"""The allocation-free XUV entry point must give what svdlinear_forward gives.

Kept in a file of its own that pytest collects last, so a run that stops at the first failure
has already exercised every other test.  It serves callers that cannot allocate device memory
when they call (all memory already owned by a framework's allocator, or a no-allocation rule
after start-up): the intermediate lives in a fixed array inside the library, shared by all calls,
so the second call below also checks that stale contents of that array are cleared.
"""
import pytest
import torch

from paper_2510_25977_b200 import binding, inputs

import _gpu

pytestmark = pytest.mark.gpu


def _case(seed, T, n_in, n_out, r):
    V = inputs.normal_tensor(seed, 0, (r, n_in), scale=n_in ** -0.5, device="cuda")
    U = inputs.normal_tensor(seed, 1, (n_out, r), scale=r ** -0.5, device="cuda")
    X = inputs.activations(T, n_in, seed=seed, device="cuda")
    return X, U, V


def test_noalloc_matches_workspace_entry_point_twice_in_a_row(oracle):
    _gpu.require_gpu()
    # the last case fills the built-in array exactly (32 x 1024 = 32768 values)
    for seed, (T, n_in, n_out, r) in enumerate([(8, 512, 1408, 64), (27, 264, 696, 40), (32, 512, 704, 1024)]):
        X, U, V = _case(20 + seed, T, n_in, n_out, r)
        Y_ref = binding.svdlinear_forward(X, U, V)
        Y = torch.full((T, n_out), 5.0, dtype=torch.bfloat16, device="cuda")  # caller-owned output
        free_before = torch.cuda.mem_get_info()[0]
        binding.svdlinear_forward_noalloc(X, U, V, Y)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before  # nothing was allocated on the device
        ref = Y_ref.double()
        delta = (Y.double() - ref).abs()
        assert delta.max() <= _gpu.MAX_REL * ref.abs().max()
        assert delta.sum() <= _gpu.MEAN_REL * ref.abs().sum()
        # and against the oracle, with the same tolerances as every other parity test
        _gpu.assert_close(Y, oracle.svdlinear(X, U, V), f"noalloc call {seed}")


def test_noalloc_rejects_sizes_beyond_the_fixed_scratch():
    _gpu.require_gpu()
    X, U, V = _case(30, 8, 256, 256, 64)
    Y = torch.empty((8, 256), dtype=torch.bfloat16, device="cuda")
    L = binding.lib()
    too_many_tokens = L.svdlinear_forward_noalloc(X.data_ptr(), binding.NOALLOC_MAX_T + 1, 256, 256, 64, U.data_ptr(),
                                                  V.data_ptr(), Y.data_ptr(), None)
    too_wide = L.svdlinear_forward_noalloc(X.data_ptr(), 32, 256, 256, 2048, U.data_ptr(), V.data_ptr(), Y.data_ptr(), None)
    assert too_many_tokens == -2 and too_wide == -2
    # T * r within the array, but the rank's strip of Z would not fit the second kernel's shared memory:
    # refused on the host, before the clear or any kernel is enqueued (the output stays untouched)
    Y.fill_(7.0)
    torch.cuda.synchronize()
    for T, r in [(4, 8192), (1, 32768), (1, binding.NOALLOC_MAX_R + 8)]:
        assert L.svdlinear_forward_noalloc(X.data_ptr(), T, 256, 256, r, U.data_ptr(), V.data_ptr(), Y.data_ptr(), None) == -2
    torch.cuda.synchronize()
    assert bool((Y == 7.0).all())
    assert "unsupported" in binding.strerror(-2)
