"""Element-by-element parity of the CUDA path with the oracle on a reduced model (several tiles, ragged tails)."""
import numpy as np
import pytest

from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import percache as pcb
from paper_2601_11553_b200 import workloads as wl
from tests import gpu_helpers as G
from tests import helpers as H

pytestmark = pytest.mark.gpu


def run_case(w: wl.Workload, flags: int, check_store: bool = True):
    # RMSNorm gains drawn away from 1: a gain that is dropped, swapped between the two norms or mis-indexed must fail
    weights = wl.make_weights(w.shape, w.seed, random_gains=True)
    model = H.oracle_model(w.shape, weights)
    ids_lens = {c: l for p in w.prompts for c, l in zip(p.chunk_ids, p.chunk_len)}
    store = G.oracle_store_alone(model, w.seed, [(c, ids_lens[c]) for c in w.cached_ids])
    want = orc.reuse_prefill(model, store, [H.oracle_prompt(p, [i for i, c in enumerate(p.chunk_ids) if c in w.cached_ids])
                                            for p in w.prompts], keep_ctx=True)
    # the assembled context is checked bit for bit below, so this pass must assemble one
    with G.make_handle(w.shape, weights, w.prompts, flags=flags | pcb.FLAG_ALWAYS_GATHER) as h:
        # the oracle committed the misses: push only what was cached before the call
        G.push_store(h, store, w.cached_ids)
        got = h.prefill(G.specs_for(w.prompts, w.cached_ids))
        G.check_plan(h.read_plan(), [r.layout for r in want])
        G.check_ctx(h, want, range(w.shape.n_layers))
        stats = []
        for b, (g, r) in enumerate(zip(got, want)):
            assert g.n_total == r.layout.n_total and g.n_new == len(r.layout.new_slots)
            assert np.array_equal(g.hit_mask, r.layout.hit_mask)
            c = G.compare_hidden(g.out_hidden, r.out_hidden)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (b, c)
            stats.append(c)
        if check_store:
            # missed chunks are now stored: bf16 K/V within one bf16 step of the oracle's slices
            for p in w.prompts:
                for cid, n in zip(p.chunk_ids, p.chunk_len):
                    assert h.has_chunk(cid) == n
                    if cid in w.cached_ids:
                        continue
                    k, v = h.get_chunk_kv(cid)
                    for got_bits, want_f in ((k, store.kv[cid][0]), (v, store.kv[cid][1])):
                        gf = orc.bf16_bits_to_f64(got_bits).reshape(want_f.shape)
                        step = 2.0 ** (np.floor(np.log2(np.maximum(np.maximum(np.abs(want_f), np.abs(gf)), 2.0 ** -20))) - 7)
                        # layer 0 depends on the token alone: the fp16 operand rounding of the normed input
                        # moves the sum by ~1e-3 at most, then the bf16 rounding may fall one step apart;
                        # deeper layers inherit the hidden-state tolerance
                        assert np.all(np.abs(gf[0] - want_f[0]) <= 1.001 * step[0] + 2e-3)
                        assert np.max(np.abs(gf - want_f)) <= G.TOL_MAX_ABS
                        assert np.mean(np.abs(gf - want_f)) <= G.TOL_MEAN_ABS
        return stats


CASES = [
    dict(seed=41, n_layers=1, chunk_lens=[128, 128, 128], n_query=32, hit_idx=[0, 1, 2]),
    dict(seed=42, n_layers=2, chunk_lens=[100, 152, 37], n_query=21, hit_idx=[1]),
    dict(seed=43, n_layers=3, chunk_lens=[16, 200, 5, 130], n_query=1, hit_idx=[0, 2]),
    dict(seed=44, n_layers=2, chunk_lens=[300, 140], n_query=70, hit_idx=[]),
]


@pytest.mark.parametrize("case", CASES, ids=lambda c: f"seed{c['seed']}")
@pytest.mark.parametrize("flags", [pcb.FLAG_REFERENCE_KERNELS, pcb.FLAG_REFERENCE_ATTENTION, 0],
                         ids=["plain-kernels", "umma-gemm+plain-attn", "umma"])
def test_small_model_parity(case, flags):
    run_case(wl.small_workload(**case), flags)


def test_wide_model_uses_the_two_pass_norm():
    """d_model above 2048 takes the RMSNorm kernel that walks the row twice; gains are random here as well."""
    w = wl.small_workload(seed=49, n_layers=2, chunk_lens=[96, 40], n_query=33, hit_idx=[0], d_model=2304)
    run_case(w, 0)


def test_all_hits_no_query_rows_is_rejected_or_empty():
    """A prompt whose every chunk hits and that has no query has no new rows: the call succeeds with n_new = 0."""
    w = wl.small_workload(seed=45, n_layers=1, chunk_lens=[48, 20], n_query=0, hit_idx=[0, 1])
    weights = wl.make_weights(w.shape, w.seed)
    model = H.oracle_model(w.shape, weights)
    store = G.oracle_store_alone(model, w.seed, list(zip(w.prompts[0].chunk_ids, w.prompts[0].chunk_len)))
    with G.make_handle(w.shape, weights, w.prompts) as h:
        G.push_store(h, store, w.cached_ids)
        p = w.prompts[0]
        got = h.prefill([pcb.PromptSpec(p.chunk_ids, p.chunk_len, None, None, 0)])
        assert got[0].n_new == 0 and got[0].n_total == 68 and got[0].hit_mask.tolist() == [1, 1]


def test_batch_of_ragged_prompts_and_first_miss_wins():
    shape = wl.small_workload(seed=46, n_layers=2, chunk_lens=[8], n_query=1, hit_idx=[]).shape
    weights = wl.make_weights(shape, 46, random_gains=True)
    model = H.oracle_model(shape, weights)
    mk = lambda cid, n: wl.chunk_hidden_for(46, cid, n, shape.d_model)
    prompts = [
        wl.Prompt([100, 101], [40, 130], 17, [mk(100, 40), mk(101, 130)], wl.make_hidden(46, (2, 0), 17, shape.d_model)),
        wl.Prompt([101, 102, 100], [130, 33, 40], 5, [mk(101, 130), mk(102, 33), mk(100, 40)],
                  wl.make_hidden(46, (2, 1), 5, shape.d_model)),
        wl.Prompt([103], [64], 129, [mk(103, 64)], wl.make_hidden(46, (2, 2), 129, shape.d_model)),
    ]
    store = G.oracle_store_alone(model, 46, [(103, 64)])
    want = orc.reuse_prefill(model, store, [H.oracle_prompt(p, [0] if p.chunk_ids[0] == 103 else []) for p in prompts],
                             keep_ctx=True)
    with G.make_handle(shape, weights, prompts) as h:
        G.push_store(h, store, [103])
        got = h.prefill(G.specs_for(prompts, [103]))
        G.check_plan(h.read_plan(), [r.layout for r in want])
        G.check_ctx(h, want, range(shape.n_layers))
        for g, r in zip(got, want):
            c = G.compare_hidden(g.out_hidden, r.out_hidden)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, c
        # chunk 101 is kept as prompt 0 computed it (in-context K/V differ between the two prompts at layer 1)
        k, _ = h.get_chunk_kv(101)
        kf = orc.bf16_bits_to_f64(k).reshape(store.kv[101][0].shape)
        assert np.mean(np.abs(kf - store.kv[101][0])) < 2e-3
        # second call: everything hits; query rows repeat the first call's (idempotence)
        again = h.prefill(G.specs_for(prompts, [100, 101, 102, 103]))
        for a, g, p in zip(again, got, prompts):
            assert a.hit_mask.tolist() == [1] * len(p.chunk_ids) and a.n_new == p.n_query
        # prompt 0's chunks were stored from prompt 0 itself: its query rows must reproduce closely
        assert np.max(np.abs(again[0].out_hidden - got[0].out_hidden[-17:])) < 2e-2


def test_many_units_of_every_length_in_one_call():
    """One call whose attention work list holds units of one block and of many, tiles of one row and of 128, several
    items per CTA and units cut along the context: what the two MMA-issuing threads of the attention kernel hand to
    each other (S buffer, P, PV completion) is exercised across every kind of unit boundary."""
    shape = wl.small_workload(seed=47, n_layers=2, chunk_lens=[8], n_query=1, hit_idx=[]).shape
    weights = wl.make_weights(shape, 47, random_gains=True)
    model = H.oracle_model(shape, weights)
    lens = {200 + c: int(n) for c, n in enumerate([5, 16, 33, 64, 100, 128, 129, 200, 257, 400, 48, 7])}
    mk = lambda cid: wl.chunk_hidden_for(47, cid, lens[cid], shape.d_model)
    cached = [201, 204, 207, 209]
    prompts = []
    for b, (ids, nq) in enumerate([([200], 1), ([201, 202], 3), ([209, 203], 128), ([204, 205, 206], 40),
                                   ([207], 300), ([208, 210], 17), ([209, 207, 204], 1), ([211, 201], 129),
                                   ([205], 64), ([206, 209, 208], 2)]):
        prompts.append(wl.Prompt(ids, [lens[c] for c in ids], nq, [mk(c) for c in ids],
                                 wl.make_hidden(47, (2, b), nq, shape.d_model)))
    store = G.oracle_store_alone(model, 47, [(c, lens[c]) for c in cached])
    want = orc.reuse_prefill(model, store, [H.oracle_prompt(p, [i for i, c in enumerate(p.chunk_ids) if c in cached])
                                            for p in prompts], commit=False)
    with G.make_handle(shape, weights, prompts) as h:
        G.push_store(h, store, cached)
        got = h.prefill(G.specs_for(prompts, cached))
        G.check_plan(h.read_plan(), [r.layout for r in want])
        for b, (g, r) in enumerate(zip(got, want)):
            assert g.n_new == len(r.layout.new_slots)
            c = G.compare_hidden(g.out_hidden, r.out_hidden)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (b, c)


def test_host_side_errors_leave_store_unchanged():
    w = wl.small_workload(seed=47, n_layers=1, chunk_lens=[32, 32], n_query=4, hit_idx=[])
    weights = wl.make_weights(w.shape, w.seed)
    p = w.prompts[0]
    with G.make_handle(w.shape, weights, w.prompts, pool_pages=3) as h:
        def code(fn):
            with pytest.raises(pcb.PerCacheError) as e:
                fn()
            return e.value.code
        spec = G.specs_for(w.prompts, [])[0]
        # 4 pages needed, 3 in the pool
        assert code(lambda: h.prefill([spec])) == pcb.E_NOSPACE
        assert h.has_chunk(p.chunk_ids[0]) is None and h.stats()["pages_free"] == 3
        # miss without input
        no_in = pcb.PromptSpec(p.chunk_ids, p.chunk_len, [None, None], p.query_hidden)
        assert code(lambda: h.prefill([no_in])) == pcb.E_MISS_NO_INPUT
        # over capacity
        big = pcb.PromptSpec([9], [4096], [np.zeros((4096, w.shape.d_model), np.uint16)], p.query_hidden)
        assert code(lambda: h.prefill([big])) == pcb.E_CAPACITY
        assert code(lambda: h.prefill([spec, spec])) == pcb.E_CAPACITY
        # put / duplicate / length mismatch / drop
        kz = np.zeros((1, 32, w.shape.kv_dim), np.uint16)
        h.put_chunk_kv(p.chunk_ids[0], kz, kz)
        assert code(lambda: h.put_chunk_kv(p.chunk_ids[0], kz, kz)) == pcb.E_EXISTS
        bad = pcb.PromptSpec([p.chunk_ids[0]], [31], [None], p.query_hidden)
        assert code(lambda: h.prefill([bad])) == pcb.E_LEN_MISMATCH
        assert h.stats()["pages_free"] == 1
        h.drop_chunk(p.chunk_ids[0])
        assert h.stats()["pages_free"] == 3
        assert code(lambda: h.drop_chunk(p.chunk_ids[0])) == pcb.E_NOTFOUND


def test_synthetic_pool_values_match_generator():
    w = wl.small_workload(seed=48, n_layers=2, chunk_lens=[40], n_query=1, hit_idx=[])
    weights = wl.make_weights(w.shape, w.seed)
    with G.make_handle(w.shape, weights, w.prompts) as h:
        h.put_chunk_synthetic(777, 40, 3)
        k, v = h.get_chunk_kv(777)
        for l in range(2):
            assert np.array_equal(k[l], wl.pool_kv_values(3, 777, 0, l, 40, w.shape.kv_dim))
            assert np.array_equal(v[l], wl.pool_kv_values(3, 777, 1, l, 40, w.shape.kv_dim))
