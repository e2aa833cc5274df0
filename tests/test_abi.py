"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and refuses to compute without a GPU."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2601_11553_b200 import percache as pcb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "percache.h")).read()
    return sorted(set(re.findall(r"PERCACHE_API\s+[\w\s\*]+?\b(percache_\w+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2601_11553_b200 import build
    build.build()
    return pcb.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 14
    assert set(names) == set(pcb.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_strerror(lib):
    assert lib.percache_strerror(0) == b"ok"
    for code in range(-10, 0):
        assert lib.percache_strerror(code) not in (b"", b"unknown error")
    assert lib.percache_strerror(-99) == b"unknown error"


def test_struct_sizes_match_header():
    # natural alignment of the declarations in percache.h
    assert C.sizeof(pcb.Config) == 96
    assert C.sizeof(pcb.LayerWeights) == 72
    assert C.sizeof(pcb.PromptStruct) == 64
    assert C.sizeof(pcb.ResultStruct) == 40
    assert C.sizeof(pcb.StatsStruct) == 192


def test_argument_validation_needs_no_gpu(lib):
    out = C.c_void_p()
    assert lib.percache_create(None, None, 0, C.byref(out)) == pcb.E_INVAL
    cfg = pcb.Config(1, 256, 4, 2, 64, 512, 1e6, 1e-6, 16, 8, 64, 1, 64, 64, 0, None, 0)   # head_dim 64: unsupported
    lw = (pcb.LayerWeights * 1)()
    assert lib.percache_create(C.byref(cfg), lw, 0, C.byref(out)) == pcb.E_INVAL
    assert lib.percache_destroy(None) == pcb.OK
    assert lib.percache_has_chunk(None, 1, None) == pcb.E_INVAL
    assert lib.percache_prefill(None, None, 0, None) == pcb.E_INVAL


def test_no_cpu_fallback(lib):
    """Without a CUDA device the library fails loudly instead of computing anywhere else."""
    torch = pytest.importorskip("torch")
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    a = np.zeros((128, 64), dtype=np.float16)
    with pytest.raises(pcb.PerCacheError) as e:
        pcb.debug_gemm(a, a)
    assert e.value.code == pcb.E_CUDA
    with pytest.raises(pcb.PerCacheError) as e:
        pcb.debug_gemm(a, a, use_reference=True)
    assert e.value.code == pcb.E_CUDA


def test_dependent_data_is_not_read_through_read_only_loads():
    """Kernels run beside their producer (programmatic launch), so what the producer writes must not be read with
    __ldg or through a const __restrict__ pointer: such a load may be scheduled above griddepcontrol.wait.  The
    buffers that are written by one kernel of a step and read by the next are checked by name."""
    src_dir = os.path.join(os.path.dirname(pcb.__file__), "csrc")
    produced = ["partial_o", "partial_ml", "kctx", "vctx", "attn_out", "resid", "qbuf"]
    for name in ("attn_umma.cu", "attn_decode.cu", "gemm_small.cu", "gemm_umma.cu"):
        text = open(os.path.join(src_dir, name)).read()
        for buf in produced:
            assert not re.search(r"__ldg\([^;]*\b%s\b" % buf, text), (name, buf)
            assert not re.search(r"const\s+\w+\s*\*\s*__restrict__\s+%s\b" % buf, text), (name, buf)
    norm = open(os.path.join(src_dir, "kernels_mem.cu")).read()
    for kernel in ("rmsnorm_kernel", "rmsnorm_long_kernel"):
        sig = norm[norm.index("%s(" % kernel):]
        sig = sig[:sig.index(")")]
        assert "__restrict__ x" not in sig, kernel
