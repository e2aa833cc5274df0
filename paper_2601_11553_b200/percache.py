"""Thin ctypes binding of libpercache.so: argument marshalling only.

Every step of reuse-prefill runs inside the CUDA library; this module converts
Python objects to the pointers and structs of ``include/percache.h`` and back.
Host buffers are numpy arrays (bf16 as ``uint16`` bit patterns); device buffers
are anything with ``data_ptr()`` and ``is_cuda`` (torch tensors).

The library is built in-tree by ``python -m paper_2601_11553_b200.build``.  If it
is missing, importing this module works but every use raises ``PerCacheError``;
there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Any, Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpercache.so")

OK = 0
E_INVAL, E_NOMEM, E_NOSPACE, E_EXISTS, E_LEN_MISMATCH = -1, -2, -3, -4, -5
E_MISS_NO_INPUT, E_CAPACITY, E_DEVICE_TIMEOUT, E_CUDA, E_NOTFOUND = -6, -7, -8, -9, -10
FLAG_REFERENCE_KERNELS, FLAG_PHASE_TIMING, FLAG_REFERENCE_ATTENTION, FLAG_EVICT_LFU = 1, 2, 4, 8
FLAG_SINGLE_CTA_GEMM = 16
FLAG_NO_SMALL_ROW_KERNELS = 32
FLAG_PAPER_MODE = 64
FLAG_GATHER_FREE, FLAG_ALWAYS_GATHER = 128, 256
PAGE_TOKENS = 16
PHASES = ("gather", "norm", "qkv", "attn", "oproj", "gateup", "down", "io")
EXPORTS = ("percache_create", "percache_destroy", "percache_put_chunk_kv", "percache_prefill",
           "percache_has_chunk", "percache_drop_chunk", "percache_get_chunk_kv", "percache_get_chunk_q", "percache_put_chunk_synthetic",
           "percache_get_stats", "percache_set_flags", "percache_decode", "percache_set_decode_reserve", "percache_set_store_limit", "percache_chunk_info", "percache_debug_read_plan", "percache_debug_read_ctx", "percache_debug_attn_plan",
           "percache_debug_gemm", "percache_debug_gemm_noalloc", "percache_debug_capture_layers", "percache_debug_wait_probe", "percache_path_key", "percache_qa_top1", "percache_strerror")


class PerCacheError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {_strerror(code)} ({code})")
        self.code = code


class Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("d_ffn", C.c_int32),
                ("rope_theta", C.c_float), ("rms_eps", C.c_float), ("page_tokens", C.c_int32),
                ("pool_pages", C.c_int64), ("max_prompt_tokens", C.c_int32), ("max_batch_prompts", C.c_int32),
                ("max_batch_ctx_tokens", C.c_int64), ("max_batch_new_rows", C.c_int64), ("device", C.c_int32),
                ("stream", C.c_void_p), ("flags", C.c_uint32)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")]


class PromptStruct(C.Structure):
    _fields_ = [("n_chunks", C.c_int32), ("chunk_ids", C.POINTER(C.c_uint64)), ("chunk_len", C.POINTER(C.c_int32)),
                ("chunk_hidden", C.POINTER(C.c_void_p)), ("n_query", C.c_int32), ("query_hidden", C.c_void_p),
                ("hidden_on_device", C.c_int32), ("match_mode", C.c_int32), ("reuse_tail_drop", C.c_int32)]


class ResultStruct(C.Structure):
    _fields_ = [("out_hidden", C.c_void_p), ("out_capacity_rows", C.c_int64), ("out_on_device", C.c_int32),
                ("hit_mask", C.POINTER(C.c_uint8)), ("n_new", C.c_int32), ("n_total", C.c_int32)]


class StatsStruct(C.Structure):
    _fields_ = [("n_prompts", C.c_int32), ("chunks_hit", C.c_int32), ("chunks_missed", C.c_int32),
                ("ctx_tokens", C.c_int64), ("hit_tokens", C.c_int64), ("new_rows", C.c_int64),
                ("pages_used", C.c_int64), ("pages_free", C.c_int64), ("host_plan_us", C.c_double),
                ("device_us", C.c_double), ("phase_us", C.c_double * len(PHASES)),
                ("phase_launches", C.c_int32 * len(PHASES)), ("attn_visible_pairs", C.c_int64), ("evictions", C.c_int64),
                ("gather_free", C.c_int32), ("reserved0", C.c_int32)]


_lib = None


def load_library() -> C.CDLL:
    """dlopen libpercache.so and declare the prototypes of include/percache.h."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise PerCacheError(E_CUDA, f"{LIB_PATH} is missing (build it: python -m paper_2601_11553_b200.build)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64
    lib.percache_create.argtypes = [C.POINTER(Config), C.POINTER(LayerWeights), i32, C.POINTER(vp)]
    lib.percache_destroy.argtypes = [vp]
    lib.percache_put_chunk_kv.argtypes = [vp, u64, i32, vp, vp, i32]
    lib.percache_prefill.argtypes = [vp, C.POINTER(PromptStruct), i32, C.POINTER(ResultStruct)]
    lib.percache_decode.argtypes = [vp, i32, vp, i32, vp, i32]
    lib.percache_set_decode_reserve.argtypes = [vp, i32]
    lib.percache_has_chunk.argtypes = [vp, u64, C.POINTER(i32)]
    lib.percache_drop_chunk.argtypes = [vp, u64]
    lib.percache_get_chunk_kv.argtypes = [vp, u64, vp, vp]
    lib.percache_get_chunk_q.argtypes = [vp, u64, vp]
    lib.percache_put_chunk_synthetic.argtypes = [vp, u64, i32, u64]
    lib.percache_get_stats.argtypes = [vp, C.POINTER(StatsStruct)]
    lib.percache_set_flags.argtypes = [vp, C.c_uint32]
    lib.percache_set_store_limit.argtypes = [vp, i64]
    lib.percache_chunk_info.argtypes = [vp, u64, C.POINTER(i32), C.POINTER(i64)]
    lib.percache_debug_read_plan.argtypes = [vp, i32, C.POINTER(i32), i64]
    lib.percache_debug_read_plan.restype = i64
    lib.percache_debug_read_ctx.argtypes = [vp, i32, i32, vp, vp, i64]
    lib.percache_debug_attn_plan.argtypes = [vp, i32, i32, i32, i32, vp, i64, vp]
    lib.percache_debug_gemm.argtypes = [i32, i32, i32, i32, vp, vp, vp, i32]
    lib.percache_debug_gemm_noalloc.argtypes = [i32, i32, i32, i32, vp, vp, vp]
    lib.percache_debug_capture_layers.argtypes = [vp, vp, i64]
    lib.percache_debug_wait_probe.argtypes = [i32, C.c_uint32, C.POINTER(i32), C.POINTER(u64)]
    lib.percache_qa_top1.argtypes = [i32, vp, vp, i32, i32, vp, i32, C.c_float, vp, vp, vp, C.POINTER(C.c_float)]
    lib.percache_path_key.argtypes = [C.POINTER(u64), i32]
    lib.percache_path_key.restype = u64
    lib.percache_strerror.argtypes = [C.c_int]
    lib.percache_strerror.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("percache_debug_read_plan", "percache_strerror", "percache_path_key"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _strerror(code: int) -> str:
    try:
        return load_library().percache_strerror(code).decode()
    except Exception:
        return "library not loaded"


def _is_device(x: Any) -> bool:
    return hasattr(x, "data_ptr") and bool(getattr(x, "is_cuda", False))


def _ptr(x: Any) -> int:
    """Address of a contiguous numpy array or torch tensor."""
    if x is None:
        return 0
    if hasattr(x, "data_ptr"):
        if not x.is_contiguous():
            raise ValueError("tensor must be contiguous")
        return int(x.data_ptr())
    a = x
    if not isinstance(a, np.ndarray) or not a.flags["C_CONTIGUOUS"]:
        raise ValueError("expected a C-contiguous numpy array")
    return int(a.ctypes.data)


def _check(rc: int, what: str) -> None:
    if rc != OK:
        raise PerCacheError(rc, what)


@dataclass
class PromptSpec:
    """One prompt: chunk ids, their lengths, bf16 hidden states of chunks (None where a hit is expected) and of the query."""
    chunk_ids: Sequence[int]
    chunk_len: Sequence[int]
    chunk_hidden: Optional[Sequence[Any]]        # each: [len, d] uint16 numpy (bf16 bits) or device bf16 tensor, or None
    query_hidden: Any                            # [n_query, d]
    n_query: Optional[int] = None
    match_prefix: bool = False                   # True: PERCACHE_MATCH_PREFIX_PATH (the paper's prefix-tree walk)
    tail_drop: int = 0                           # reuse_tail_drop (prefix matching only)


@dataclass
class PromptResult:
    out_hidden: Any          # float32 [n_new, d]: numpy (host) or the caller's device tensor slice
    hit_mask: np.ndarray     # uint8 [n_chunks]
    n_new: int
    n_total: int


class PerCache:
    """Handle of one model on one GPU (wraps percache_create / percache_destroy)."""

    def __init__(self, *, n_layers: int, d_model: int, n_q_heads: int, n_kv_heads: int, head_dim: int, d_ffn: int,
                 weights: Sequence[Dict[str, Any]], pool_pages: int, max_prompt_tokens: int,
                 max_batch_prompts: int = 1, max_batch_ctx_tokens: Optional[int] = None,
                 max_batch_new_rows: Optional[int] = None, rope_theta: float = 1.0e6, rms_eps: float = 1.0e-6,
                 device: int = 0, stream: int = 0, flags: int = 0):
        self._lib = load_library()
        self._h = C.c_void_p()
        self.d_model = d_model
        self.n_layers = n_layers
        self.kv_dim = n_kv_heads * head_dim
        self.q_dim = n_q_heads * head_dim
        self.paper_mode = bool(flags & FLAG_PAPER_MODE)
        if max_batch_ctx_tokens is None:
            max_batch_ctx_tokens = max_prompt_tokens * max_batch_prompts
        if max_batch_new_rows is None:
            max_batch_new_rows = max_batch_ctx_tokens
        cfg = Config(n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, rope_theta, rms_eps, PAGE_TOKENS,
                     pool_pages, max_prompt_tokens, max_batch_prompts, max_batch_ctx_tokens, max_batch_new_rows,
                     device, C.c_void_p(stream or None), flags)
        if len(weights) != n_layers:
            raise ValueError("one weight dict per layer")
        on_dev = _is_device(weights[0]["wq"])
        lw = (LayerWeights * n_layers)()
        for l, w in enumerate(weights):
            for name, _ in LayerWeights._fields_:
                if _is_device(w[name]) != on_dev:
                    raise ValueError("weights must be all host or all device")
                setattr(lw[l], name, _ptr(w[name]))
        _check(self._lib.percache_create(C.byref(cfg), lw, 1 if on_dev else 0, C.byref(self._h)), "percache_create")

    # ------------------------------------------------------------------ lifetime
    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.percache_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # ------------------------------------------------------------------ store
    def put_chunk_kv(self, chunk_id: int, k: Any, v: Any) -> None:
        """k, v: bf16 [n_layers, n_tokens, n_kv_heads*head_dim] (uint16 numpy bits, or device bf16 tensors)."""
        n_tokens = int(k.shape[1])
        _check(self._lib.percache_put_chunk_kv(self._h, chunk_id, n_tokens, _ptr(k), _ptr(v), 1 if _is_device(k) else 0),
               "percache_put_chunk_kv")

    def put_chunk_synthetic(self, chunk_id: int, n_tokens: int, seed: int) -> None:
        _check(self._lib.percache_put_chunk_synthetic(self._h, chunk_id, n_tokens, seed), "percache_put_chunk_synthetic")

    def has_chunk(self, chunk_id: int) -> Optional[int]:
        n = C.c_int32(-1)
        rc = self._lib.percache_has_chunk(self._h, chunk_id, C.byref(n))
        if rc == E_NOTFOUND:
            return None
        _check(rc, "percache_has_chunk")
        return int(n.value)

    def set_store_limit(self, pages: int) -> None:
        _check(self._lib.percache_set_store_limit(self._h, pages), "percache_set_store_limit")

    def chunk_info(self, chunk_id: int):
        """(n_tokens, retrieval count) of a stored chunk, or None."""
        n, r = C.c_int32(-1), C.c_int64(-1)
        rc = self._lib.percache_chunk_info(self._h, chunk_id, C.byref(n), C.byref(r))
        if rc == E_NOTFOUND:
            return None
        _check(rc, "percache_chunk_info")
        return int(n.value), int(r.value)

    def drop_chunk(self, chunk_id: int) -> None:
        _check(self._lib.percache_drop_chunk(self._h, chunk_id), "percache_drop_chunk")

    def get_chunk_kv(self, chunk_id: int):
        n = self.has_chunk(chunk_id)
        if n is None:
            raise PerCacheError(E_NOTFOUND, "percache_get_chunk_kv")
        k = np.empty((self.n_layers, n, self.kv_dim), dtype=np.uint16)
        v = np.empty_like(k)
        _check(self._lib.percache_get_chunk_kv(self._h, chunk_id, _ptr(k), _ptr(v)), "percache_get_chunk_kv")
        return k, v

    def get_chunk_q(self, chunk_id: int) -> np.ndarray:
        """Paper-faithful mode: the node's cached Q, bf16 bits [n_layers, n_tokens, n_q_heads*head_dim]."""
        n = self.has_chunk(chunk_id)
        if n is None:
            raise PerCacheError(E_NOTFOUND, "percache_get_chunk_q")
        q = np.empty((self.n_layers, n, self.q_dim), dtype=np.uint16)
        _check(self._lib.percache_get_chunk_q(self._h, chunk_id, _ptr(q)), "percache_get_chunk_q")
        return q

    # ------------------------------------------------------------------ prefill
    def prefill(self, prompts: Sequence[PromptSpec], out: Optional[Sequence[Any]] = None) -> List[PromptResult]:
        """percache_prefill.  `out[b]`: optional caller buffer float32 [rows >= n_new, d] (numpy or device tensor)."""
        n = len(prompts)
        ps = (PromptStruct * n)()
        rs = (ResultStruct * n)()
        keep: List[Any] = []
        outs: List[Any] = []
        masks: List[np.ndarray] = []
        for b, p in enumerate(prompts):
            nc = len(p.chunk_ids)
            ids = (C.c_uint64 * max(nc, 1))(*[int(c) for c in p.chunk_ids])
            lens = (C.c_int32 * max(nc, 1))(*[int(c) for c in p.chunk_len])
            hid = (C.c_void_p * max(nc, 1))()
            on_dev = _is_device(p.query_hidden) if p.query_hidden is not None else False
            if p.chunk_hidden is not None:
                for i in range(nc):
                    hcur = p.chunk_hidden[i] if i < len(p.chunk_hidden) else None
                    if hcur is not None:
                        if p.query_hidden is None:
                            on_dev = _is_device(hcur)
                        elif _is_device(hcur) != on_dev:
                            raise ValueError("hidden states of one prompt must be all host or all device")
                        hid[i] = _ptr(hcur)
            nq = int(p.n_query if p.n_query is not None else (0 if p.query_hidden is None else p.query_hidden.shape[0]))
            ps[b] = PromptStruct(nc, ids, lens, hid, nq, _ptr(p.query_hidden) if nq > 0 else None, 1 if on_dev else 0,
                                 1 if p.match_prefix else 0, int(p.tail_drop))
            keep += [ids, lens, hid]
            if out is not None and out[b] is not None:
                ob = out[b]
            else:
                ob = np.empty((int(sum(p.chunk_len)) + nq, self.d_model), dtype=np.float32)
            mask = np.zeros(max(nc, 1), dtype=np.uint8)
            rs[b] = ResultStruct(_ptr(ob), int(ob.shape[0]), 1 if _is_device(ob) else 0,
                                 mask.ctypes.data_as(C.POINTER(C.c_uint8)), 0, 0)
            outs.append(ob)
            masks.append(mask)
        _check(self._lib.percache_prefill(self._h, ps, n, rs), "percache_prefill")
        # rows that come back: the new rows, or every row of the prompt in the paper-faithful mode
        n_out = [int(rs[b].n_total if self.paper_mode else rs[b].n_new) for b in range(n)]
        return [PromptResult(outs[b][: n_out[b]], masks[b][: len(prompts[b].chunk_ids)], int(rs[b].n_new),
                             int(rs[b].n_total)) for b in range(n)]

    # ------------------------------------------------------------------ introspection
    def set_decode_reserve(self, tokens_per_prompt: int) -> None:
        """Keep this many context slots free behind every prompt of later prefill calls (for decode)."""
        _check(self._lib.percache_set_decode_reserve(self._h, int(tokens_per_prompt)), "percache_set_decode_reserve")

    def decode(self, hidden: Any, out: Optional[Any] = None):
        """percache_decode: one token per prompt of the last prefill call.

        hidden: bf16 [n_prompts, d_model] as a uint16/bf16 numpy array (host) or a torch device tensor.
        Returns fp32 [n_prompts, d_model] (numpy), or fills and returns `out` (host numpy or device tensor).
        """
        n = int(hidden.shape[0])
        if out is None:
            out = np.empty((n, self.d_model), dtype=np.float32)
        _check(self._lib.percache_decode(self._h, n, _ptr(hidden), 1 if _is_device(hidden) else 0, _ptr(out),
                                         1 if _is_device(out) else 0), "percache_decode")
        return out

    def stats(self) -> Dict[str, Any]:
        s = StatsStruct()
        _check(self._lib.percache_get_stats(self._h, C.byref(s)), "percache_get_stats")
        d = {k: getattr(s, k) for k, _ in StatsStruct._fields_ if k not in ("phase_us", "phase_launches")}
        d["phase_us"] = {PHASES[i]: s.phase_us[i] for i in range(len(PHASES))}
        d["phase_launches"] = {PHASES[i]: s.phase_launches[i] for i in range(len(PHASES))}
        return d

    def set_flags(self, flags: int) -> None:
        _check(self._lib.percache_set_flags(self._h, flags), "percache_set_flags")

    def read_plan(self) -> Dict[str, np.ndarray]:
        names = ("cu_ctx", "cu_new", "slot_chunk", "slot_offset", "slot_is_new", "row_slot")
        st = self.stats()
        cap = int(max(st["ctx_tokens"], st["new_rows"], st["n_prompts"] + 1)) + 1
        res = {}
        for which, name in enumerate(names):
            buf = np.empty(cap, dtype=np.int32)
            n = self._lib.percache_debug_read_plan(self._h, which, buf.ctypes.data_as(C.POINTER(C.c_int32)), cap)
            if n < 0:
                raise PerCacheError(int(n), "percache_debug_read_plan")
            res[name] = buf[:n].copy()
        return res

    def capture_layers(self, buf: Optional[np.ndarray]) -> None:
        """percache_debug_capture_layers: float32 host array [n_layers + 1, rows, d_model] (flat capacity counts), or
        None to switch the capture off.  The array must stay alive until then."""
        if buf is None:
            _check(self._lib.percache_debug_capture_layers(self._h, None, 0), "percache_debug_capture_layers")
            return
        if buf.dtype != np.float32 or not buf.flags["C_CONTIGUOUS"]:
            raise ValueError("capture buffer must be C-contiguous float32")
        _check(self._lib.percache_debug_capture_layers(self._h, _ptr(buf), int(buf.size)), "percache_debug_capture_layers")

    def read_ctx(self, prompt: int, layer: int, n_total: int):
        """Assembled (rotated K, V) of one prompt and layer: two float16 arrays [n_total, kv_dim]."""
        k = np.empty((n_total, self.kv_dim), dtype=np.float16)
        v = np.empty_like(k)
        _check(self._lib.percache_debug_read_ctx(self._h, prompt, layer, _ptr(k), _ptr(v), n_total),
               "percache_debug_read_ctx")
        return k, v


def debug_attn_plan(n_blocks: Sequence[int], units_per_tile: int, n_ctas: int = 148, max_partial_slots: int = 298):
    """percache_debug_attn_plan (host only): returns (items [n][6] = tile, unit, blk_begin, blk_end, partial_slot,
    cta; CTAs used; split units; estimated makespan in quarter blocks)."""
    nb = np.ascontiguousarray(np.asarray(n_blocks, dtype=np.int32))
    cap = int(len(nb)) * units_per_tile + 2 * n_ctas + 8
    items = np.zeros((cap, 6), dtype=np.int32)
    counts = np.zeros(4, dtype=np.int64)
    _check(load_library().percache_debug_attn_plan(_ptr(nb) if len(nb) else None, len(nb), units_per_tile, n_ctas,
                                                   max_partial_slots, _ptr(items), cap, _ptr(counts)),
           "percache_debug_attn_plan")
    return items[:int(counts[0])].copy(), int(counts[1]), int(counts[2]), int(counts[3])


def path_key(chunk_ids: Sequence[int]) -> int:
    """Store key of the prefix-tree node reached by the path `chunk_ids` (percache_path_key)."""
    arr = (C.c_uint64 * max(len(chunk_ids), 1))(*[int(c) for c in chunk_ids])
    return int(load_library().percache_path_key(arr, len(chunk_ids)))


def debug_gemm(a_f16: np.ndarray, b_f16: np.ndarray, use_reference: bool = False, device: int = 0,
               pair: bool = False) -> np.ndarray:
    """C = A @ B.T through the tcgen05 GEMM core (or the plain kernel, or the CTA-pair variant of the tcgen05
    GEMM): fp16 in, fp32 out, host arrays."""
    lib = load_library()
    m, k = a_f16.shape
    n = b_f16.shape[0]
    c = np.empty((m, n), dtype=np.float32)
    _check(lib.percache_debug_gemm(device, m, n, k, _ptr(np.ascontiguousarray(a_f16)), _ptr(np.ascontiguousarray(b_f16)),
                                   _ptr(c), 2 if pair else (1 if use_reference else 0)), "percache_debug_gemm")
    return c


def debug_wait_probe(limit_us: int = 1000, device: int = 0):
    """percache_debug_wait_probe: returns (return code, recorded device code, [ns waited by the two waiters])."""
    code = C.c_int32(0)
    waited = (C.c_uint64 * 2)()
    rc = load_library().percache_debug_wait_probe(device, int(limit_us), C.byref(code), waited)
    return int(rc), int(code.value), [int(waited[0]), int(waited[1])]


NOALLOC_SCRATCH_BYTES = 16 << 20


def debug_gemm_noalloc(a_f16: np.ndarray, b_f16: np.ndarray, device: int = 0) -> np.ndarray:
    """C = A @ B.T through the tcgen05 GEMM without any device allocation (percache_debug_gemm_noalloc).

    For callers that cannot call cudaMalloc: the device copies live in a fixed 16 MiB array inside the
    library; larger problems raise PerCacheError(E_CAPACITY).  Calls must not overlap on the GPU.
    """
    lib = load_library()
    m, k = a_f16.shape
    n = b_f16.shape[0]
    c = np.empty((m, n), dtype=np.float32)
    _check(lib.percache_debug_gemm_noalloc(device, m, n, k, _ptr(np.ascontiguousarray(a_f16)),
                                           _ptr(np.ascontiguousarray(b_f16)), _ptr(c)), "percache_debug_gemm_noalloc")
    return c


def qa_top1(bank: Any, queries: Any, tau_query: float, device: int = 0, stream: int = 0, timing: bool = False):
    """percache_qa_top1: bank [n, dim] and queries [q, dim] are fp32 device tensors; returns (index, score, hit)
    arrays, plus the kernel time in microseconds when timing is set."""
    n, dim = int(bank.shape[0]), int(bank.shape[1])
    nq = int(queries.shape[0])
    idx = np.empty(nq, dtype=np.int32)
    score = np.empty(nq, dtype=np.float32)
    hit = np.empty(nq, dtype=np.uint8)
    us = C.c_float(0.0)
    _check(load_library().percache_qa_top1(device, C.c_void_p(stream or None), _ptr(bank), n, dim, _ptr(queries), nq,
                                           C.c_float(tau_query), _ptr(idx), _ptr(score), _ptr(hit),
                                           C.byref(us) if timing else None), "percache_qa_top1")
    return (idx, score, hit, float(us.value)) if timing else (idx, score, hit)
