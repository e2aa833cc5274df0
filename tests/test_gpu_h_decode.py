"""Decode steps after a reuse-prefill, through the C ABI, against the decode oracle."""
import numpy as np
import pytest

from oracle import decode as dec
from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import percache as pcb
from paper_2601_11553_b200 import workloads as wl
from tests import gpu_helpers as G
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _decode_case(seed, n_layers, prompts_spec, n_steps, reserve, flags=0, **model_kw):
    """prompts_spec: list of (chunk_lens, n_query, hit_idx).  Returns nothing; asserts parity at every step."""
    ws = [wl.small_workload(seed=seed, n_layers=n_layers, chunk_lens=cl, n_query=nq, hit_idx=hi, id_base=100 + 50 * b,
                            **model_kw)
          for b, (cl, nq, hi) in enumerate(prompts_spec)]
    shape = ws[0].shape
    weights = wl.make_weights(shape, seed, random_gains=True)     # the small-row projections fold the norm in
    model = H.oracle_model(shape, weights)
    prompts = [w.prompts[0] for w in ws]
    cached = [c for w in ws for c in w.cached_ids]
    lens = {c: l for p in prompts for c, l in zip(p.chunk_ids, p.chunk_len)}
    store = G.oracle_store_alone(model, seed, [(c, lens[c]) for c in cached])
    want = orc.reuse_prefill(model, store, [H.oracle_prompt(p, [i for i, c in enumerate(p.chunk_ids) if c in cached])
                                            for p in prompts], keep_ctx=True, commit=False)
    states = [dec.begin_decode(r) for r in want]
    toks = [wl.make_hidden(seed, (9, j), len(prompts), shape.d_model) for j in range(n_steps)]   # bf16 bits [B, d]
    with G.make_handle(shape, weights, prompts, decode_reserve=reserve, flags=flags) as h:
        h.set_decode_reserve(reserve)
        G.push_store(h, store, cached)
        got = h.prefill(G.specs_for(prompts, cached))
        for b, r in enumerate(want):
            c = G.compare_hidden(got[b].out_hidden, r.out_hidden)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, c
        for j in range(n_steps):
            out = h.decode(np.ascontiguousarray(toks[j]))
            ref = np.stack([dec.decode_step(model, states[b], orc.bf16_bits_to_f64(toks[j][b]))
                            for b in range(len(prompts))])
            c = G.compare_hidden(out, ref)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (j, c)
        # the appended K/V: V is the bf16-rounded projection (a format conversion away from the oracle's),
        # K its rotation to the token's position
        for b, st in enumerate(states):
            n_total = want[b].layout.n_total
            k, v = h.read_ctx(b, shape.n_layers - 1, n_total + n_steps)
            wk = st.k_ctx[-1].reshape(n_total + n_steps, -1)
            wv = st.v_ctx[-1].reshape(n_total + n_steps, -1)
            assert np.max(np.abs(v[n_total:].astype(np.float64) - wv[n_total:])) < 3e-2
            assert np.max(np.abs(k[n_total:].astype(np.float64) - wk[n_total:])) < 3e-2
            # and the prefill part of the context is untouched by the decode steps
            assert np.array_equal(v[:n_total][want[b].layout.slot_is_new == 0].view(np.uint16),
                                  wv[:n_total][want[b].layout.slot_is_new == 0].astype(np.float16).view(np.uint16))
        # one step more than the reserve is refused and changes nothing
        for _ in range(reserve - n_steps):
            h.decode(np.ascontiguousarray(toks[0]))
        with pytest.raises(pcb.PerCacheError) as e:
            h.decode(np.ascontiguousarray(toks[0]))
        assert e.value.code == pcb.E_CAPACITY


def test_decode_single_prompt_two_layers():
    _decode_case(seed=61, n_layers=2, prompts_spec=[([128, 100, 160], 40, [0, 2])], n_steps=3, reserve=4)


def test_decode_crosses_a_context_block_boundary():
    # 250 + 5 = 255 tokens: the second decoded token is the first slot of the third 128-slot block
    _decode_case(seed=62, n_layers=1, prompts_spec=[([250], 5, [0])], n_steps=3, reserve=3)


def test_decode_batch_of_ragged_prompts():
    _decode_case(seed=63, n_layers=2, prompts_spec=[([64, 37], 9, [1]), ([300], 17, []), ([16, 16, 16], 1, [0, 1, 2])],
                 n_steps=2, reserve=2)


def test_decode_six_prompts():
    # five to eight rows take the eight-row variant of the weight-streaming kernels
    spec = [([48], 3 + b, [0] if b % 2 else []) for b in range(6)]
    _decode_case(seed=65, n_layers=2, prompts_spec=spec, n_steps=2, reserve=2)


def test_decode_ten_prompts_uses_the_tensor_core_path():
    spec = [([32 + 16 * (b % 3)], 2 + b, [0] if b % 3 == 0 else []) for b in range(10)]
    _decode_case(seed=66, n_layers=2, prompts_spec=spec, n_steps=2, reserve=2)


def test_decode_single_prompt_on_the_tensor_core_path():
    _decode_case(seed=61, n_layers=2, prompts_spec=[([128, 100, 160], 40, [0, 2])], n_steps=2, reserve=2,
                 flags=pcb.FLAG_NO_SMALL_ROW_KERNELS)


def test_decode_four_query_heads_per_kv_head():
    # two head pairs per KV head in the prefill attention, the four-head variant of the decode attention
    _decode_case(seed=67, n_layers=2, prompts_spec=[([200, 90], 21, [0]), ([130], 7, [])], n_steps=2, reserve=2,
                 n_q_heads=8, n_kv_heads=2, d_model=512)


def test_decode_needs_the_batch_of_the_last_prefill():
    w = wl.small_workload(seed=64, n_layers=1, chunk_lens=[32], n_query=4, hit_idx=[])
    weights = wl.make_weights(w.shape, w.seed)
    with G.make_handle(w.shape, weights, w.prompts, decode_reserve=2) as h:
        tok = wl.make_hidden(64, (9, 0), 2, w.shape.d_model)
        with pytest.raises(pcb.PerCacheError):           # nothing prefilled yet
            h.decode(np.ascontiguousarray(tok[:1]))
        h.set_decode_reserve(2)
        h.prefill(G.specs_for(w.prompts, []))
        with pytest.raises(pcb.PerCacheError):           # two rows for a batch of one prompt
            h.decode(np.ascontiguousarray(tok))
        h.decode(np.ascontiguousarray(tok[:1]))


def test_decode_after_the_28_layer_workload_at_full_size():
    """Two decode steps behind the full-depth, 2112-token prompt (three of eight chunks cached), in the launch
    configuration the benchmark's decode workload times."""
    w = wl.config1()
    weights = wl.make_weights(w.shape, w.seed)
    model = H.oracle_model(w.shape, weights)
    p = w.prompts[0]
    lens = dict(zip(p.chunk_ids, p.chunk_len))
    store = G.oracle_store_alone(model, w.seed, [(c, lens[c]) for c in w.cached_ids])
    cached = set(w.cached_ids)
    want = orc.reuse_prefill(model, store, [H.oracle_prompt(p, [i for i, c in enumerate(p.chunk_ids) if c in cached])],
                             keep_ctx=True, commit=False)[0]
    st = dec.begin_decode(want)
    toks = wl.make_hidden(w.seed, (9, 0), 2, w.shape.d_model)
    with G.make_handle(w.shape, weights, w.prompts, decode_reserve=2) as h:
        h.set_decode_reserve(2)
        G.push_store(h, store, w.cached_ids)
        got = h.prefill(G.specs_for(w.prompts, w.cached_ids))[0]
        c = G.compare_hidden(got.out_hidden, want.out_hidden)
        assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, c
        for j in range(2):
            out = h.decode(np.ascontiguousarray(toks[j:j + 1]))
            ref = dec.decode_step(model, st, orc.bf16_bits_to_f64(toks[j]))
            c = G.compare_hidden(out[0], ref)
            print("decode step", j, c)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (j, c)
