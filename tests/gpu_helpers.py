"""Helpers for the GPU parity tests: run one workload through the C ABI and through the oracle."""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import percache as pcb
from paper_2601_11553_b200 import workloads as wl
from tests import helpers as H

TOL_MAX_ABS = 3e-2      # final hidden states, stated with the workloads
TOL_MEAN_ABS = 3e-3


def make_handle(shape: wl.ModelShape, weights: List[dict], prompts: Sequence[wl.Prompt], pool_pages: int = 0,
                flags: int = 0, slack_prompts: int = 0, decode_reserve: int = 0) -> pcb.PerCache:
    max_t = max(p.n_total for p in prompts) + decode_reserve
    total = sum(p.n_total for p in prompts) + decode_reserve * len(prompts)
    if pool_pages <= 0:
        pool_pages = sum((l + 15) // 16 for p in prompts for l in p.chunk_len) + 64
    return pcb.PerCache(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                        n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn, weights=weights,
                        pool_pages=pool_pages, max_prompt_tokens=max_t, max_batch_prompts=len(prompts) + slack_prompts,
                        max_batch_ctx_tokens=total, max_batch_new_rows=total, rope_theta=shape.rope_theta,
                        rms_eps=shape.rms_eps, flags=flags)


def specs_for(prompts: Sequence[wl.Prompt], cached: Sequence[int]) -> List[pcb.PromptSpec]:
    cached = set(cached)
    out = []
    for p in prompts:
        hid = None
        if p.chunk_hidden:
            hid = [None if c in cached else h for c, h in zip(p.chunk_ids, p.chunk_hidden)]
        out.append(pcb.PromptSpec(list(p.chunk_ids), list(p.chunk_len), hid, p.query_hidden, p.n_query))
    return out


def oracle_store_alone(model: orc.Model, seed: int, ids_lens: Sequence[Tuple[int, int]]) -> orc.Store:
    """Cache content made by prefilling every chunk alone (no hits, no query)."""
    store = orc.Store()
    for cid, n in ids_lens:
        H.populate_alone(model, store, seed, cid, n)
    return store


def push_store(handle: pcb.PerCache, store: orc.Store, ids: Sequence[int]) -> None:
    """Give the library exactly the oracle's cached K/V (bf16 bits)."""
    for cid in ids:
        k, v = store.kv[cid]
        L, n = k.shape[0], k.shape[1]
        handle.put_chunk_kv(cid, np.ascontiguousarray(orc.f64_to_bf16_bits(k).reshape(L, n, -1)),
                            np.ascontiguousarray(orc.f64_to_bf16_bits(v).reshape(L, n, -1)))


def f16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of fp16 at |x| (normal range), at least the subnormal spacing."""
    ax = np.maximum(np.abs(x.astype(np.float64)), 2.0 ** -14)
    return 2.0 ** (np.floor(np.log2(ax)) - 10)


def compare_hidden(got: np.ndarray, want: np.ndarray) -> Dict[str, float]:
    d = np.abs(got.astype(np.float64) - want)
    return {"max_abs": float(d.max()) if d.size else 0.0, "mean_abs": float(d.mean()) if d.size else 0.0}


def check_plan(plan: Dict[str, np.ndarray], layouts: Sequence[orc.Layout]) -> None:
    """Index assembly must match the oracle's layout bit for bit."""
    cu_ctx = np.cumsum([0] + [l.n_total for l in layouts]).astype(np.int32)
    cu_new = np.cumsum([0] + [len(l.new_slots) for l in layouts]).astype(np.int32)
    assert np.array_equal(plan["cu_ctx"], cu_ctx)
    assert np.array_equal(plan["cu_new"], cu_new)
    assert np.array_equal(plan["slot_chunk"], np.concatenate([l.slot_chunk for l in layouts]))
    assert np.array_equal(plan["slot_offset"], np.concatenate([l.slot_offset for l in layouts]))
    assert np.array_equal(plan["slot_is_new"], np.concatenate([l.slot_is_new for l in layouts]).astype(np.int32))
    assert np.array_equal(plan["row_slot"], np.concatenate([l.new_slots for l in layouts]))


def check_ctx(handle: pcb.PerCache, results: Sequence[orc.PromptResult], layers: Sequence[int]) -> Dict[str, float]:
    """Assembled context against the oracle's: hit slots' V bit-exact, rotated K within 1 fp16 ulp of the pair."""
    worst = 0.0
    for b, res in enumerate(results):
        lay = res.layout
        hit = lay.slot_is_new == 0
        for l in layers:
            k, v = handle.read_ctx(b, l, lay.n_total)
            kv_dim = k.shape[1]
            want_v = res.v_ctx[l].reshape(lay.n_total, kv_dim)
            want_k = res.k_ctx[l].reshape(lay.n_total, kv_dim)
            # gathered V: a pure format conversion of identical stored values -> identical bits
            assert np.array_equal(v[hit].view(np.uint16), want_v[hit].astype(np.float16).view(np.uint16)), \
                f"gathered V differs (prompt {b}, layer {l})"
            if hit[0]:     # position 0: rotation by zero, K is a pure copy as well
                assert np.array_equal(k[0].view(np.uint16), want_k[0].astype(np.float16).view(np.uint16))
            # rotated K of hit slots: 1 ulp at the magnitude of the rotated pair
            kk = k[hit].astype(np.float64).reshape(-1, kv_dim // 128, 2, 64)
            ww = want_k[hit].reshape(-1, kv_dim // 128, 2, 64)
            mag = np.maximum(np.abs(ww[:, :, 0]), np.abs(ww[:, :, 1]))[:, :, None, :]
            err = np.abs(kk - ww) / f16_ulp(np.broadcast_to(mag, ww.shape))
            worst = max(worst, float(err.max()) if err.size else 0.0)
            assert err.size == 0 or err.max() <= 1.0 + 1e-6, f"rotated K off by {err.max()} ulp (prompt {b}, layer {l})"
    return {"k_rot_max_ulp": worst}


# --------------------------------------------------------------------------- teacher-forced, sampled-row checks
def layout_only_store(ids_lens: Dict[int, int], cached: Sequence[int], shape: wl.ModelShape) -> orc.Store:
    """A store that knows which chunks are cached and how long they are, without holding any tensor (the arrays
    are zero-strided views): enough for the oracle's layout step at sizes where the tensors would not fit."""
    st = orc.Store()
    for c in cached:
        z = np.broadcast_to(np.float64(0.0), (shape.n_layers, ids_lens[c], shape.n_kv_heads, shape.head_dim))
        st.kv[c] = (z, z)
    return st


def sample_rows(layout: orc.Layout, n_random: int, rng: np.random.Generator) -> np.ndarray:
    """Row indices (into the prompt's new rows): the first and last row of every run of consecutive new slots,
    plus n_random others."""
    new = layout.new_slots
    m = new.shape[0]
    if m == 0:
        return np.zeros(0, dtype=np.int64)
    brk = np.nonzero(np.diff(new) != 1)[0]
    picks = set([0, m - 1] + [int(i) for i in brk] + [int(i) + 1 for i in brk])
    rest = np.setdiff1d(np.arange(m), np.fromiter(picks, dtype=np.int64))
    if n_random > 0 and rest.size:
        picks.update(int(i) for i in rng.choice(rest, size=min(n_random, rest.size), replace=False))
    return np.array(sorted(picks), dtype=np.int64)


def teacher_forced_check(w: wl.Workload, layers: Sequence[int], n_random_per_prompt: int, flags: int = 0,
                         random_gains: bool = False) -> Dict[str, float]:
    """Full-size, full-depth parity where a whole oracle run is out of reach.

    The library runs the workload once, handing out the residual stream as it enters every block.  For each
    checked block the oracle gets the library's own input of that block (all new rows: the block's K and V depend
    on every one of them), forms the block's output for sampled rows, and that is compared with the library's
    input of the next block.  Blocks are then independent, so any subset can be checked; what an error in block l
    does to later blocks is outside this check (end-to-end runs at full depth cover that on the smaller workloads).
    Cached chunks hold the seeded integer pool values on both sides.
    """
    shape = w.shape
    weights = wl.make_weights(shape, w.seed, random_gains=random_gains)
    model = H.oracle_model(shape, weights)
    ids_lens = {c: l for p in w.prompts for c, l in zip(p.chunk_ids, p.chunk_len)}
    cached = set(w.cached_ids)
    lstore = layout_only_store(ids_lens, w.cached_ids, shape)
    oprompts = [H.oracle_prompt(p, [i for i, c in enumerate(p.chunk_ids) if c in cached]) for p in w.prompts]
    layouts = [orc.assemble_layout(lstore, op) for op in oprompts]
    m_total = sum(len(l.new_slots) for l in layouts)
    cap = np.empty((shape.n_layers + 1, m_total, shape.d_model), dtype=np.float32)
    with make_handle(shape, weights, w.prompts, flags=flags) as h:
        for c in w.cached_ids:
            h.put_chunk_synthetic(c, ids_lens[c], w.seed)
        h.capture_layers(cap)
        got = h.prefill(specs_for(w.prompts, w.cached_ids))
        h.capture_layers(None)
        check_plan(h.read_plan(), layouts)
        stats = h.stats()
    cu = np.cumsum([0] + [len(l.new_slots) for l in layouts])
    for b, g in enumerate(got):        # the last capture is the call's output
        assert np.array_equal(g.out_hidden, cap[shape.n_layers, cu[b]:cu[b + 1]])
    rng = np.random.default_rng([w.seed, 7010])
    rows_of = [sample_rows(l, n_random_per_prompt, rng) for l in layouts]
    hkv, hd = shape.n_kv_heads, shape.head_dim
    worst = {"max_abs": 0.0, "mean_abs": 0.0, "rows_per_layer": int(sum(r.size for r in rows_of)),
             "layers": list(layers), "device_us": stats["device_us"]}
    for l in layers:
        pool: Dict[int, tuple] = {}

        def seg(c):       # this layer's stored K, V of chunk c (the integer pool values), generated once per layer
            if c not in pool:
                n = ids_lens[c]
                pool[c] = tuple(orc.bf16_bits_to_f64(wl.pool_kv_values(w.seed, c, which, l, n, hkv * hd)).reshape(n, hkv, hd)
                                for which in (0, 1))
            return pool[c]
        errs = []
        for b, (p, lay) in enumerate(zip(w.prompts, layouts)):
            if rows_of[b].size == 0:
                continue
            segs, start = [], 0
            for i, (c, n) in enumerate(zip(p.chunk_ids, p.chunk_len)):
                if lay.hit_mask[i]:
                    segs.append((start,) + seg(c))
                start += n
            x = cap[l, cu[b]:cu[b + 1]].astype(np.float64)
            want, _, _ = orc.block_rows(model, l, x, lay.new_slots, lay.n_total, segs, rows_of[b])
            errs.append(np.abs(cap[l + 1, cu[b] + rows_of[b]].astype(np.float64) - want))
        e = np.concatenate(errs)
        worst["max_abs"] = max(worst["max_abs"], float(e.max()))
        worst["mean_abs"] = max(worst["mean_abs"], float(e.mean()))
        assert e.max() <= TOL_MAX_ABS and e.mean() <= TOL_MEAN_ABS, (w.name, l, float(e.max()), float(e.mean()))
    return worst
