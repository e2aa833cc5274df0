"""Parity of the CUDA path with the oracle on the five workload shapes (full size where the oracle
finishes in about a minute, reduced depth otherwise), in the launch configuration the benchmark times."""
import numpy as np
import pytest

from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import percache as pcb
from paper_2601_11553_b200 import workloads as wl
from tests import gpu_helpers as G
from tests import helpers as H

pytestmark = pytest.mark.gpu


def run_workload(w: wl.Workload, ctx_layers=None, random_gains=False):
    weights = wl.make_weights(w.shape, w.seed, random_gains=random_gains)
    model = H.oracle_model(w.shape, weights)
    ids_lens = {c: l for p in w.prompts for c, l in zip(p.chunk_ids, p.chunk_len)}
    if w.cache_source == "integer_pool":
        store = orc.Store()
        hkv, hd = w.shape.n_kv_heads, w.shape.head_dim
        for c in w.cached_ids:
            n = ids_lens[c]
            k = np.stack([orc.bf16_bits_to_f64(wl.pool_kv_values(w.seed, c, 0, l, n, hkv * hd)).reshape(n, hkv, hd)
                          for l in range(w.shape.n_layers)])
            v = np.stack([orc.bf16_bits_to_f64(wl.pool_kv_values(w.seed, c, 1, l, n, hkv * hd)).reshape(n, hkv, hd)
                          for l in range(w.shape.n_layers)])
            store.put(c, k, v)
    else:
        store = G.oracle_store_alone(model, w.seed, [(c, ids_lens[c]) for c in w.cached_ids])
    cached = set(w.cached_ids)
    want = orc.reuse_prefill(model, store, [H.oracle_prompt(p, [i for i, c in enumerate(p.chunk_ids) if c in cached])
                                            for p in w.prompts], keep_ctx=True, commit=False)
    layers = list(range(w.shape.n_layers)) if ctx_layers is None else ctx_layers
    # the assembled context is compared bit for bit, so the contiguous context must be built here; the gather-free
    # form of the same workloads is checked in test_gpu_l_gather_free.py and, at full size, by the teacher-forced tests
    with G.make_handle(w.shape, weights, w.prompts, flags=pcb.FLAG_ALWAYS_GATHER) as h:
        if w.cache_source == "integer_pool":
            for c in w.cached_ids:
                h.put_chunk_synthetic(c, ids_lens[c], w.seed)
        else:
            G.push_store(h, store, w.cached_ids)
        got = h.prefill(G.specs_for(w.prompts, w.cached_ids))
        G.check_plan(h.read_plan(), [r.layout for r in want])
        ctx = G.check_ctx(h, want, layers)
        worst = {"max_abs": 0.0, "mean_abs": 0.0}
        for g, r in zip(got, want):
            assert np.array_equal(g.hit_mask, r.layout.hit_mask)
            c = G.compare_hidden(g.out_hidden, r.out_hidden)
            worst = {k: max(worst[k], c[k]) for k in worst}
        print(w.name, worst, ctx, h.stats()["device_us"])
        assert worst["max_abs"] <= G.TOL_MAX_ABS and worst["mean_abs"] <= G.TOL_MEAN_ABS, worst
        return worst


def test_config0_single_layer_all_hits():
    run_workload(wl.config0())


def test_config1_28_layers_bernoulli_hits():
    run_workload(wl.config1(), ctx_layers=[0, 1, 13, 27])


def test_config2_shape_two_layers():
    w = wl.config2()
    w.shape = wl.ModelShape(n_layers=2, **wl.SHAPE_B)
    run_workload(w, random_gains=True)


def test_config3_shape_batched_ragged_zipf_pool():
    w = wl.config3(n_prompts=12, pool=256, n_layers=2)
    run_workload(w)


def test_config4_shape_long_context_90pct_hits():
    w = wl.config4(0.9)
    w.shape = wl.ModelShape(n_layers=2, **wl.SHAPE_A)
    run_workload(w, random_gains=True)
