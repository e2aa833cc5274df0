"""The allocation-free GEMM entry point against the allocating one, through the C ABI.

Some users of the library cannot allocate device memory when they call it: their process has given the
whole GPU to another allocator, or they sit in a serving loop where cudaMalloc's device-wide
synchronisation is not acceptable.  percache_debug_gemm_noalloc serves them from a fixed array inside
the library.  The array keeps the previous call's bytes, so the test makes two calls in a row, the second
one smaller and with a ragged row count, and checks each against percache_debug_gemm.
"""
import numpy as np
import pytest
import torch

from paper_2601_11553_b200 import percache as pcb


@pytest.mark.gpu
def test_noalloc_gemm_matches_allocating_gemm_twice_in_a_row():
    rng = np.random.default_rng(2024)
    for call, (m, n, k) in enumerate(((300, 384, 1024), (37, 256, 128))):
        a = (rng.standard_normal((m, k)) * 0.5).astype(np.float16)
        b = (rng.standard_normal((n, k)) * 0.5).astype(np.float16)
        want = pcb.debug_gemm(a, b)
        free_before = torch.cuda.mem_get_info(0)[0]
        got = pcb.debug_gemm_noalloc(a, b)
        # The second call must leave the device's free memory untouched.  (The first call of a process is where the
        # CUDA runtime loads the part of the library image that holds the fixed array, so free memory drops once there.)
        if call == 1:
            assert torch.cuda.mem_get_info(0)[0] == free_before
        exact = a.astype(np.float64) @ b.astype(np.float64).T
        tol = max(4e-7 * k * 0.25 + 1e-6, 2e-4 * np.sqrt(k) * 0.25)      # the GEMM tests' tolerance
        assert np.max(np.abs(got - exact)) < tol
        assert np.max(np.abs(got - want)) < tol
        assert np.array_equal(got, want)      # same kernel, same tiles: same bits


@pytest.mark.gpu
def test_noalloc_gemm_rejects_what_does_not_fit():
    a = np.zeros((4096, 4096), dtype=np.float16)
    with pytest.raises(pcb.PerCacheError) as e:
        pcb.debug_gemm_noalloc(a, a)
    assert e.value.code == pcb.E_CAPACITY
    # a row count near the top of the int32 range must be refused by the size check, not wrap around in it
    one = np.zeros((1, 64), dtype=np.float16)
    lib = pcb.load_library()
    c = np.zeros(1, dtype=np.float32)
    assert lib.percache_debug_gemm_noalloc(0, 2**31 - 1, 128, 64, one.ctypes.data, one.ctypes.data, c.ctypes.data) == pcb.E_CAPACITY
