"""The paper's prefix-tree matching (PERCACHE_MATCH_PREFIX_PATH) through the C ABI: a sequence of queries whose
chunk lists share prefixes.  Hits must be exactly the matched prefix, results must match the oracle in the same
mode — and therefore full prefill without any cache, which the oracle equals in this mode (pinned on the CPU)."""
import numpy as np
import pytest

from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import percache as pcb
from paper_2601_11553_b200 import workloads as wl
from tests import gpu_helpers as G
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_prefix_tree_sequence():
    shape = wl.small_workload(seed=71, n_layers=3, chunk_lens=[16], n_query=1, hit_idx=[]).shape
    weights = wl.make_weights(shape, 71, random_gains=True)
    model = H.oracle_model(shape, weights)
    lens = {1: 130, 5: 100, 7: 37, 9: 152, 12: 64}
    hid = {c: wl.chunk_hidden_for(71, c, n, shape.d_model) for c, n in lens.items()}
    queries = [([1, 5, 7], [0, 0, 0]), ([1, 5, 9], [1, 1, 0]), ([1, 5, 9, 12], [1, 1, 1, 0]), ([5, 1], [0, 0]),
               ([1, 5, 7], [1, 1, 1]), ([1, 9], [1, 0])]
    store = orc.Store()
    h = pcb.PerCache(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                     n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn, weights=weights,
                     pool_pages=256, max_prompt_tokens=600, max_batch_prompts=1)
    with h:
        for qi, (ids, want_mask) in enumerate(queries):
            qh = wl.make_hidden(71, (2, qi), 20 + qi, shape.d_model)
            want = orc.reuse_prefill(model, store, [orc.Prompt(ids, [lens[c] for c in ids],
                                                               [orc.bf16_bits_to_f64(hid[c]) for c in ids],
                                                               orc.bf16_bits_to_f64(qh))], match_prefix=True)[0]
            got = h.prefill([pcb.PromptSpec(ids, [lens[c] for c in ids], [hid[c] for c in ids], qh,
                                            match_prefix=True)])[0]
            assert got.hit_mask.tolist() == want_mask == want.layout.hit_mask.tolist(), qi
            G.check_plan(h.read_plan(), [want.layout])
            c = G.compare_hidden(got.out_hidden, want.out_hidden)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (qi, c)
            # and against plain full prefill of the whole prompt
            full, _, _ = orc.dense_prefill(model, np.concatenate([orc.bf16_bits_to_f64(hid[c]) for c in ids] +
                                                                 [orc.bf16_bits_to_f64(qh)]))
            c = G.compare_hidden(got.out_hidden, full[want.layout.new_slots])
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (qi, c)
        # nodes are stored under their path keys, not under plain ids
        assert h.has_chunk(pcb.path_key([1, 5, 9, 12])) == lens[12]
        assert h.has_chunk(pcb.path_key([5, 1])) == lens[1]
        assert h.has_chunk(pcb.path_key([1])) == lens[1]
        assert h.has_chunk(1) is None and h.has_chunk(pcb.path_key([9])) is None
        # an evicted ancestor ends the walk: its stored descendants are recomputed, not reused, and not stored twice
        h.drop_chunk(pcb.path_key([1, 5]))
        qh = wl.make_hidden(71, (2, 99), 9, shape.d_model)
        got = h.prefill([pcb.PromptSpec([1, 5, 9], [lens[c] for c in (1, 5, 9)], [hid[c] for c in (1, 5, 9)], qh,
                                        match_prefix=True)])[0]
        assert got.hit_mask.tolist() == [1, 0, 0]
        assert h.has_chunk(pcb.path_key([1, 5])) == lens[5]


@pytest.mark.parametrize("drop", [1, 16, 37, 100])
def test_tail_of_the_final_matched_chunk_is_recomputed(drop):
    """reuse_tail_drop (paper Appendix B, tokenisation paragraph): the last tokens of the final matched chunk are new
    rows computed from their inputs; layout bit-exact, hidden states within tolerance of the oracle and of plain
    full prefill, nothing stored twice.  Cases: one token, one whole page, a ragged count, the whole chunk."""
    shape = wl.small_workload(seed=72, n_layers=2, chunk_lens=[16], n_query=1, hit_idx=[]).shape
    weights = wl.make_weights(shape, 72, random_gains=True)
    model = H.oracle_model(shape, weights)
    lens = {1: 130, 5: 100, 9: 48}
    hid = {c: wl.chunk_hidden_for(72, c, n, shape.d_model) for c, n in lens.items()}
    qh = wl.make_hidden(72, (2, 0), 19, shape.d_model)
    f64 = orc.bf16_bits_to_f64
    store = orc.Store()
    h = pcb.PerCache(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                     n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn, weights=weights,
                     pool_pages=64, max_prompt_tokens=400, max_batch_prompts=1, flags=pcb.FLAG_ALWAYS_GATHER)
    with h:
        warm = [1, 5]
        orc.reuse_prefill(model, store, [orc.Prompt(warm, [lens[c] for c in warm], [f64(hid[c]) for c in warm],
                                                    np.zeros((0, shape.d_model)))], match_prefix=True)
        # the library gets exactly the oracle's nodes (same bf16 bits), under their path keys, so that gathered
        # bytes can be compared bit for bit
        for path, (ck, cv) in store.kv.items():
            L, n = ck.shape[0], ck.shape[1]
            h.put_chunk_kv(pcb.path_key(list(path)), np.ascontiguousarray(orc.f64_to_bf16_bits(ck).reshape(L, n, -1)),
                           np.ascontiguousarray(orc.f64_to_bf16_bits(cv).reshape(L, n, -1)))
        pages_before = h.stats()["pages_used"]
        ids = [1, 5, 9]
        want = orc.reuse_prefill(model, store, [orc.Prompt(ids, [lens[c] for c in ids], [None, f64(hid[5]), f64(hid[9])],
                                                           f64(qh), tail_drop=drop)], match_prefix=True,
                                 keep_ctx=True, commit=False)[0]
        got = h.prefill([pcb.PromptSpec(ids, [lens[c] for c in ids], [None, hid[5], hid[9]], qh, match_prefix=True,
                                        tail_drop=drop)])[0]
        assert got.hit_mask.tolist() == [1, 1, 0] == want.layout.hit_mask.tolist()
        assert got.n_new == drop + lens[9] + 19 and got.n_total == 297
        G.check_plan(h.read_plan(), [want.layout])
        G.check_ctx(h, [want], range(shape.n_layers))
        c = G.compare_hidden(got.out_hidden, want.out_hidden)
        assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, c
        full, _, _ = orc.dense_prefill(model, np.concatenate([f64(hid[c]) for c in ids] + [f64(qh)]))
        c = G.compare_hidden(got.out_hidden, full[want.layout.new_slots])
        assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, c
        # only chunk 9's node was added
        assert h.stats()["pages_used"] == pages_before + 3 and h.has_chunk(pcb.path_key(ids)) == 48
        # outside prefix matching the field must be zero
        with pytest.raises(pcb.PerCacheError) as e:
            h.prefill([pcb.PromptSpec([77], [16], [hid[9][:16]], qh, tail_drop=1)])
        assert e.value.code == pcb.E_INVAL
