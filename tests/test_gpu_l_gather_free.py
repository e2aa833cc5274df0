"""The gather-free form of percache_prefill against the oracle and against the form that assembles a context.

In this form the attention reads K and V where the store keeps them (16-token pages reached through the prompt's
page table), rotates K as it loads it, and nothing is copied into a contiguous context.  The result is defined by
the same oracle; the one numeric difference is that P and V enter the second attention product as bf16."""
import numpy as np
import pytest

from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import percache as pcb
from paper_2601_11553_b200 import workloads as wl
from tests import gpu_helpers as G
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _both_forms(w: wl.Workload, match_prefix=False, tail_drop=0, extra_prompts=()):
    weights = wl.make_weights(w.shape, w.seed, random_gains=True)
    model = H.oracle_model(w.shape, weights)
    prompts = list(w.prompts) + list(extra_prompts)
    ids_lens = {c: l for p in prompts for c, l in zip(p.chunk_ids, p.chunk_len)}
    cached = set(w.cached_ids)
    store = G.oracle_store_alone(model, w.seed, [(c, ids_lens[c]) for c in w.cached_ids])
    want = orc.reuse_prefill(model, store, [H.oracle_prompt(p, [i for i, c in enumerate(p.chunk_ids) if c in cached])
                                            for p in prompts], commit=False)
    outs, kvs = {}, {}
    for form, flag in (("gather", pcb.FLAG_ALWAYS_GATHER), ("gather_free", pcb.FLAG_GATHER_FREE)):
        with G.make_handle(w.shape, weights, prompts, flags=flag) as h:
            G.push_store(h, store, w.cached_ids)
            free_before = h.stats()["pages_free"]
            got = h.prefill(G.specs_for(prompts, w.cached_ids))
            st = h.stats()
            assert st["gather_free"] == (1 if form == "gather_free" else 0)
            G.check_plan(h.read_plan(), [r.layout for r in want])          # the integer plan is the same in both forms
            stored_now = sum((ids_lens[c] + 15) // 16 for c in ids_lens if c not in cached)
            assert st["pages_free"] == free_before - stored_now              # pages lent to query rows came back
            for g, r in zip(got, want):
                assert np.array_equal(g.hit_mask, r.layout.hit_mask)
                c = G.compare_hidden(g.out_hidden, r.out_hidden)
                assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (form, c)
            outs[form] = [g.out_hidden.copy() for g in got]
            missed = [c for c in ids_lens if c not in cached]
            kvs[form] = [h.get_chunk_kv(c) for c in missed]
            if form == "gather_free":      # no contiguous context exists (and no decode reserve was set): refused
                with pytest.raises(pcb.PerCacheError) as e:
                    h.read_ctx(0, 0, want[0].layout.n_total)
                assert e.value.code == pcb.E_INVAL
                with pytest.raises(pcb.PerCacheError) as e:
                    h.decode(np.zeros((len(prompts), w.shape.d_model), np.uint16))
                assert e.value.code == pcb.E_INVAL
    for a, b in zip(outs["gather"], outs["gather_free"]):
        d = np.abs(a.astype(np.float64) - b)
        assert d.max() <= G.TOL_MAX_ABS and d.mean() <= G.TOL_MEAN_ABS
    for (ka, va), (kb, vb) in zip(kvs["gather"], kvs["gather_free"]):
        # what a missed chunk leaves in the store: block 0 depends on the token alone -> the same bits in both forms
        assert np.array_equal(ka[0], kb[0]) and np.array_equal(va[0], vb[0])
        assert np.mean(np.abs(orc.bf16_bits_to_f64(ka) - orc.bf16_bits_to_f64(kb))) <= G.TOL_MEAN_ABS
    return outs


CASES = [
    dict(seed=101, n_layers=2, chunk_lens=[128, 128, 128], n_query=32, hit_idx=[0, 1, 2]),          # all hits
    dict(seed=102, n_layers=3, chunk_lens=[64, 160, 32, 144], n_query=21, hit_idx=[0, 3]),          # hits around misses
    dict(seed=103, n_layers=2, chunk_lens=[16, 272], n_query=1, hit_idx=[1]),                       # several blocks, one query row
    dict(seed=104, n_layers=2, chunk_lens=[256, 128], n_query=150, hit_idx=[0]),                    # two row tiles
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"seed{c['seed']}")
def test_gather_free_matches_oracle_and_gather_form(case):
    _both_forms(wl.small_workload(**case))


def test_batch_of_prompts_with_shared_chunks():
    shape = wl.small_workload(seed=105, n_layers=2, chunk_lens=[16], n_query=1, hit_idx=[]).shape
    mk = lambda cid, n: wl.chunk_hidden_for(105, cid, n, shape.d_model)
    prompts = [
        wl.Prompt([100, 101], [48, 128], 17, [mk(100, 48), mk(101, 128)], wl.make_hidden(105, (2, 0), 17, shape.d_model)),
        wl.Prompt([101, 102, 100], [128, 32, 48], 5, [mk(101, 128), mk(102, 32), mk(100, 48)],
                  wl.make_hidden(105, (2, 1), 5, shape.d_model)),
        wl.Prompt([103], [64], 129, [mk(103, 64)], wl.make_hidden(105, (2, 2), 129, shape.d_model)),
    ]
    w = wl.Workload("batch105", shape, 105, prompts[:1], cached_ids=[101, 103])
    _both_forms(w, extra_prompts=prompts[1:])


def test_selection_rule():
    """Without either flag the form follows the batch: at least 8 cached tokens per new row, no prompt with more
    than 256 new rows, page-aligned chunks."""
    def form_of(chunk_lens, n_query, hit_idx, reserve=0, flags=0):
        w = wl.small_workload(seed=106, n_layers=1, chunk_lens=chunk_lens, n_query=n_query, hit_idx=hit_idx)
        weights = wl.make_weights(w.shape, w.seed)
        with G.make_handle(w.shape, weights, w.prompts, flags=flags, decode_reserve=reserve) as h:
            if reserve:
                h.set_decode_reserve(reserve)
            for c, n in zip(w.prompts[0].chunk_ids, w.prompts[0].chunk_len):
                if c in w.cached_ids:
                    h.put_chunk_synthetic(c, n, 7)
            h.prefill(G.specs_for(w.prompts, w.cached_ids))
            return h.stats()["gather_free"]
    assert form_of([128, 128], 16, [0, 1]) == 1                      # 256 cached : 16 new
    assert form_of([128, 128], 40, [0, 1]) == 0                      # 256 : 40 is below 8 : 1
    assert form_of([128, 128], 40, [0, 1], flags=pcb.FLAG_GATHER_FREE) == 1
    assert form_of([128, 128], 16, [0, 1], flags=pcb.FLAG_ALWAYS_GATHER) == 0
    assert form_of([120, 136], 16, [0, 1]) == 0                      # not page-aligned
    assert form_of([128, 128], 16, [0, 1], reserve=4) == 1           # a decode reserve does not change the choice
    assert form_of([128, 128], 16, []) == 0                          # nothing cached
    assert form_of([1024, 1024, 1024], 300, [0, 1, 2]) == 0          # 3072 : 300, but three tiles of new rows


def test_prefix_matching_with_tail_drop_gather_free():
    shape = wl.small_workload(seed=107, n_layers=2, chunk_lens=[16], n_query=1, hit_idx=[]).shape
    weights = wl.make_weights(shape, 107, random_gains=True)
    model = H.oracle_model(shape, weights)
    lens = {1: 128, 5: 96, 9: 48}
    hid = {c: wl.chunk_hidden_for(107, c, n, shape.d_model) for c, n in lens.items()}
    qh = wl.make_hidden(107, (2, 0), 19, shape.d_model)
    f64 = orc.bf16_bits_to_f64
    store = orc.Store()
    orc.reuse_prefill(model, store, [orc.Prompt([1, 5], [128, 96], [f64(hid[1]), f64(hid[5])], np.zeros((0, shape.d_model)))],
                      match_prefix=True)
    ids = [1, 5, 9]
    want = orc.reuse_prefill(model, store, [orc.Prompt(ids, [lens[c] for c in ids], [None, f64(hid[5]), f64(hid[9])],
                                                       f64(qh), tail_drop=32)], match_prefix=True, commit=False)[0]
    full, _, _ = orc.dense_prefill(model, np.concatenate([f64(hid[c]) for c in ids] + [f64(qh)]))
    h = pcb.PerCache(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                     n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn, weights=weights,
                     pool_pages=64, max_prompt_tokens=400, max_batch_prompts=1, flags=pcb.FLAG_GATHER_FREE)
    with h:
        for path, (ck, cv) in store.kv.items():
            L, n = ck.shape[0], ck.shape[1]
            h.put_chunk_kv(pcb.path_key(list(path)), np.ascontiguousarray(orc.f64_to_bf16_bits(ck).reshape(L, n, -1)),
                           np.ascontiguousarray(orc.f64_to_bf16_bits(cv).reshape(L, n, -1)))
        got = h.prefill([pcb.PromptSpec(ids, [lens[c] for c in ids], [None, hid[5], hid[9]], qh, match_prefix=True,
                                        tail_drop=32)])[0]
        assert h.stats()["gather_free"] == 1 and got.n_new == 32 + 48 + 19
        G.check_plan(h.read_plan(), [want.layout])
        for ref in (want.out_hidden, full[want.layout.new_slots]):
            c = G.compare_hidden(got.out_hidden, ref)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, c


def _decode_setup(seed, reserve, n_steps):
    from oracle import decode as dec
    ws = [wl.small_workload(seed=seed, n_layers=2, chunk_lens=cl, n_query=nq, hit_idx=hi, id_base=100 + 50 * b)
          for b, (cl, nq, hi) in enumerate([([128, 64], 9, [0, 1]), ([256], 20, [0])])]
    shape = ws[0].shape
    weights = wl.make_weights(shape, seed, random_gains=True)
    model = H.oracle_model(shape, weights)
    prompts = [w.prompts[0] for w in ws]
    cached = [c for w in ws for c in w.cached_ids]
    lens = {c: l for p in prompts for c, l in zip(p.chunk_ids, p.chunk_len)}
    store = G.oracle_store_alone(model, seed, [(c, lens[c]) for c in cached])
    want = orc.reuse_prefill(model, store, [H.oracle_prompt(p, list(range(len(p.chunk_ids)))) for p in prompts],
                             keep_ctx=True, commit=False)
    states = [dec.begin_decode(r) for r in want]
    toks = [wl.make_hidden(seed, (9, j), len(prompts), shape.d_model) for j in range(n_steps)]
    return dec, shape, weights, model, prompts, cached, store, want, states, toks


@pytest.mark.parametrize("reserve,n_steps", [(3, 3), (40, 20)])
def test_decode_after_a_gather_free_prefill_reads_the_pages(reserve, n_steps):
    """With a decode reserve the gather-free prefill keeps the pages it lent to the query rows and adds page slots for
    the tokens to come; with PERCACHE_FLAG_GATHER_FREE still set, decode steps read K and V from the pages as well (K
    rotated on load) and no context is ever assembled for the batch.  The second case decodes across page and
    128-slot block boundaries."""
    dec, shape, weights, model, prompts, cached, store, want, states, toks = _decode_setup(108, reserve, n_steps)
    with G.make_handle(shape, weights, prompts, decode_reserve=reserve, flags=pcb.FLAG_GATHER_FREE) as h:
        h.set_decode_reserve(reserve)
        G.push_store(h, store, cached)
        free_before = h.stats()["pages_free"]
        got = h.prefill(G.specs_for(prompts, cached))
        assert h.stats()["gather_free"] == 1
        lent = sum((p.n_total + reserve + 15) // 16 - sum(p.chunk_len) // 16 for p in prompts)
        assert h.stats()["pages_free"] == free_before - lent          # query rows' pages + slots for decoded tokens
        for g, r in zip(got, want):
            c = G.compare_hidden(g.out_hidden, r.out_hidden)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, c
        for j in range(n_steps):
            out = h.decode(np.ascontiguousarray(toks[j]))
            ref = np.stack([dec.decode_step(model, states[b], orc.bf16_bits_to_f64(toks[j][b])) for b in range(len(prompts))])
            c = G.compare_hidden(out, ref)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (j, c)
        with pytest.raises(pcb.PerCacheError) as e:                   # still no contiguous context
            h.read_ctx(0, 0, want[0].layout.n_total + n_steps)
        assert e.value.code == pcb.E_INVAL
        if n_steps == reserve:
            with pytest.raises(pcb.PerCacheError) as e:               # the reserve is used up
                h.decode(np.ascontiguousarray(toks[0]))
            assert e.value.code == pcb.E_CAPACITY
        # the next prefill gives the lent pages back
        h.prefill(G.specs_for(prompts[:1], cached))
        assert h.stats()["pages_free"] == free_before - ((prompts[0].n_total + reserve + 15) // 16 - sum(prompts[0].chunk_len) // 16)


@pytest.mark.parametrize("reserve_case", [0, 1], ids=["streaming-kernels", "tensor-core-kernels"])
def test_decode_after_a_gather_free_prefill_assembles_the_context_late(reserve_case):
    """Without the flag at decode time (here also with the streaming decode kernels switched off), the first decode step
    runs the fetch the prefill skipped, over every slot, which builds the context the gather form builds; the lent
    pages then go back."""
    reserve, n_steps = 3, 3
    dec, shape, weights, model, prompts, cached, store, want, states, toks = _decode_setup(109, reserve, n_steps)
    with G.make_handle(shape, weights, prompts, decode_reserve=reserve, flags=pcb.FLAG_GATHER_FREE) as h:
        h.set_decode_reserve(reserve)
        G.push_store(h, store, cached)
        free_before = h.stats()["pages_free"]
        got = h.prefill(G.specs_for(prompts, cached))
        assert h.stats()["gather_free"] == 1 and h.stats()["pages_free"] < free_before
        h.set_flags(pcb.FLAG_NO_SMALL_ROW_KERNELS if reserve_case else 0)
        for j in range(n_steps):
            out = h.decode(np.ascontiguousarray(toks[j]))
            ref = np.stack([dec.decode_step(model, states[b], orc.bf16_bits_to_f64(toks[j][b])) for b in range(len(prompts))])
            c = G.compare_hidden(out, ref)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (j, c)
            assert h.stats()["pages_free"] == free_before             # given back by the first step
        # gathered V bit for bit (the read returns the decoded tokens' slots as well)
        for b, r in enumerate(want):
            n_total = r.layout.n_total
            hit = r.layout.slot_is_new == 0
            for l in range(shape.n_layers):
                k, v = h.read_ctx(b, l, n_total + n_steps)
                want_v = r.v_ctx[l].reshape(n_total, -1)
                assert np.array_equal(v[:n_total][hit].view(np.uint16), want_v[hit].astype(np.float16).view(np.uint16))
                want_k = r.k_ctx[l].reshape(n_total, -1)
                assert np.max(np.abs(k[:n_total].astype(np.float64) - want_k)) < 3e-2
