"""tcgen05 GEMM core against float64 matmul (and the plain kernel), through the C ABI."""
import numpy as np
import pytest

from paper_2601_11553_b200 import percache as pcb

pytestmark = pytest.mark.gpu


def _inputs(m, n, k, seed):
    rng = np.random.default_rng(seed)
    a = (rng.standard_normal((m, k)) * 0.5).astype(np.float16)
    b = (rng.standard_normal((n, k)) * 0.5).astype(np.float16)
    return a, b


@pytest.mark.parametrize("m,n,k", [(128, 128, 64), (128, 128, 256), (37, 256, 128), (300, 384, 1024),
                                   (1088, 4096, 1024), (2176, 1024, 5632)])
def test_umma_gemm_matches_float64(m, n, k):
    a, b = _inputs(m, n, k, m + n + k)
    want = a.astype(np.float64) @ b.astype(np.float64).T
    got = pcb.debug_gemm(a, b)
    # fp32 accumulation of exact fp16 products: error ~ sqrt(k) * 2^-24 * |a||b|
    tol = 4e-7 * k * 0.25 + 1e-6
    assert np.max(np.abs(got - want)) < max(tol, 2e-4 * np.sqrt(k) * 0.25)
    ref = pcb.debug_gemm(a, b, use_reference=True)
    assert np.max(np.abs(ref - want)) < max(tol, 2e-4 * np.sqrt(k) * 0.25)


def test_umma_gemm_identity_layout():
    """B = identity picks columns of A: any swizzle / descriptor mistake moves elements."""
    k = n = 128
    a = (np.arange(256 * k).reshape(256, k) % 251).astype(np.float16)
    b = np.eye(n, k, dtype=np.float16)
    got = pcb.debug_gemm(a, b)
    assert np.array_equal(got, a.astype(np.float32))


@pytest.mark.parametrize("m,n,k", [(256, 256, 64), (256, 256, 512), (37, 256, 128), (300, 512, 1024),
                                   (1344, 4096, 1024), (2176, 1024, 5632), (5000, 2048, 2048)])
def test_pair_gemm_matches_float64(m, n, k):
    """The same GEMM on clusters of two CTAs (one UMMA over both CTAs' shared memory, 256 x 256 tiles)."""
    a, b = _inputs(m, n, k, m + n + k + 1)
    want = a.astype(np.float64) @ b.astype(np.float64).T
    got = pcb.debug_gemm(a, b, pair=True)
    tol = 4e-7 * k * 0.25 + 1e-6
    assert np.max(np.abs(got - want)) < max(tol, 2e-4 * np.sqrt(k) * 0.25)


def test_pair_gemm_identity_layout():
    """B = identity picks columns of A: rows 128..255 come from the second CTA, columns 128..255 from its half of B."""
    k = n = 256
    a = (np.arange(512 * k).reshape(512, k) % 251).astype(np.float16)
    b = np.eye(n, k, dtype=np.float16)
    got = pcb.debug_gemm(a, b, pair=True)
    assert np.array_equal(got, a.astype(np.float32))
