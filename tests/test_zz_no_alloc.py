"""olsgd_class_pairs_noalloc against olsgd_class_pairs, through the C ABI.

The allocation-free entry point serves callers that cannot call cudaMalloc or
cudaHostAlloc (a capture in progress on the thread, memory fully handed to a
pool, a thread that must not take the allocator's locks): it stages the table in
an array inside the library's device image.  Its output must equal the ordinary
entry point's bit for bit, on repeated calls that reuse the array.

This file sorts last on purpose, so that a run that stops at the first failure
has already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _both(lib, seed, m, device):
    stream = torch.cuda.current_stream().cuda_stream
    a = torch.full((m, 2), -1, dtype=torch.int32, device=device)
    b = torch.full((m, 2), -2, dtype=torch.int32, device=device)
    assert lib.olsgd_class_pairs(seed, m, a.data_ptr(), stream) == 0
    assert lib.olsgd_class_pairs_noalloc(seed, m, b.data_ptr(), stream) == 0
    return a.cpu().numpy(), b.cpu().numpy()


def test_noalloc_equals_allocating_entry_point_on_consecutive_calls():
    from paper_2002_09539_b200 import binding
    lib = binding.load_library()
    torch.cuda.set_device(0)
    # two calls in a row that share the scratch array, the second one smaller, so stale
    # entries of the first call sit behind the part the second call returns
    for seed, m, device in [(0, 64, "cpu"), (7, 5, "cpu"), (7, 5, "cuda"),
                            (2**63 + 11, binding.NOALLOC_MAX_WORKERS, "cpu"), (3, 1, "cpu")]:
        want, got = _both(lib, seed, m, device)
        assert np.array_equal(got, want), (seed, m, device)
        want2, got2 = _both(lib, seed + 1, m, device)
        assert np.array_equal(got2, want2)
        assert not np.array_equal(got2, got) or m == 1


def test_noalloc_matches_the_oracle_table():
    from oracle import sampling
    from paper_2002_09539_b200 import class_pairs_noalloc
    for seed, m in [(0, 64), (5, 6)]:
        assert np.array_equal(class_pairs_noalloc(seed, m).numpy(), sampling.class_pairs(seed, m))


def test_noalloc_rejects_sizes_beyond_the_fixed_array():
    from paper_2002_09539_b200 import binding
    lib = binding.load_library()
    out = torch.zeros((4, 2), dtype=torch.int32)
    stream = torch.cuda.current_stream().cuda_stream
    st = lib.olsgd_class_pairs_noalloc(0, binding.NOALLOC_MAX_WORKERS + 1, out.data_ptr(), stream)
    assert st == 1                                      # OLSGD_EINVAL, nothing launched
    assert b"exceeds the fixed scratch array" in lib.olsgd_last_error(None)
    assert lib.olsgd_class_pairs_noalloc(0, 0, out.data_ptr(), stream) == 1
    assert lib.olsgd_class_pairs_noalloc(0, 4, None, stream) == 1
    assert not out.any()
