"""Capacity management through the C ABI against the CPU model: same call sequence, same hits, same evictions,
same counters; and the numbers still match the numeric oracle when chunks come and go."""
import numpy as np
import pytest

from oracle import lfu
from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import percache as pcb
from paper_2601_11553_b200 import workloads as wl
from tests import gpu_helpers as G
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_lfu_sequence_matches_model_and_oracle():
    shape = wl.small_workload(seed=61, n_layers=2, chunk_lens=[16], n_query=1, hit_idx=[]).shape
    weights = wl.make_weights(shape, 61)
    model = H.oracle_model(shape, weights)
    rng = np.random.default_rng(61)
    lens = {cid: int(rng.integers(5, 70)) for cid in range(200, 212)}
    hidden = {cid: wl.chunk_hidden_for(61, cid, n, shape.d_model) for cid, n in lens.items()}
    limit = 9                                              # pages; single chunks take 1..5
    ref = lfu.LfuModel(limit_pages=limit)
    store = orc.Store()
    h = pcb.PerCache(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                     n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn, weights=weights,
                     pool_pages=32, max_prompt_tokens=400, max_batch_prompts=2, flags=pcb.FLAG_EVICT_LFU)
    with h:
        h.set_store_limit(limit)
        n_evicted = 0
        for call in range(14):
            n_prompts = 1 + int(rng.integers(0, 2))
            prompts = []
            for b in range(n_prompts):
                ids = [int(c) for c in rng.choice(sorted(lens), size=int(rng.integers(1, 4)), replace=False)]
                qh = wl.make_hidden(61, (2, call, b), int(rng.integers(1, 20)), shape.d_model)
                prompts.append((ids, qh))
            need = {c for ids, _ in prompts for c in ids if c not in ref.entries}
            protected = {c for ids, _ in prompts for c in ids if c in ref.entries}
            fits = sum(lfu.pages_of(lens[c]) for c in need) + sum(lfu.pages_of(ref.entries[c]["tokens"]) for c in protected) <= limit
            specs = [pcb.PromptSpec(ids, [lens[c] for c in ids], [hidden[c] for c in ids], qh) for ids, qh in prompts]
            if not fits:
                with pytest.raises(lfu.NoSpace):
                    ref.call([(ids, [lens[c] for c in ids]) for ids, _ in prompts])
                with pytest.raises(pcb.PerCacheError) as e:
                    h.prefill(specs)
                assert e.value.code == pcb.E_NOSPACE
                continue
            masks, victims = ref.call([(ids, [lens[c] for c in ids]) for ids, _ in prompts])
            for v in victims:                               # eviction precedes the computation
                store.drop(v)
            want = orc.reuse_prefill(model, store, [
                orc.Prompt(ids, [lens[c] for c in ids], [orc.bf16_bits_to_f64(hidden[c]) for c in ids],
                           orc.bf16_bits_to_f64(qh)) for ids, qh in prompts])
            got = h.prefill(specs)
            n_evicted += len(victims)
            assert h.stats()["evictions"] == len(victims)
            for g, mk, r in zip(got, masks, want):
                assert g.hit_mask.tolist() == mk == r.layout.hit_mask.tolist()
                c = G.compare_hidden(g.out_hidden, r.out_hidden)
                assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, c
            for cid in lens:
                info = h.chunk_info(cid)
                if cid in ref.entries:
                    assert info == (lens[cid], ref.entries[cid]["count"])
                else:
                    assert info is None
            assert h.stats()["pages_used"] == ref.used() <= limit
        assert n_evicted >= 3                               # the sequence really exercises eviction
        # lowering the limit evicts at once, in the model's order
        victims = ref.set_limit(4)
        h.set_store_limit(4)
        assert h.stats()["evictions"] == len(victims)
        assert sorted(c for c in lens if h.has_chunk(c) is not None) == sorted(ref.entries)


def test_without_the_flag_a_full_store_still_refuses():
    w = wl.small_workload(seed=62, n_layers=1, chunk_lens=[32, 32], n_query=2, hit_idx=[])
    weights = wl.make_weights(w.shape, w.seed)
    with G.make_handle(w.shape, weights, w.prompts, pool_pages=8) as h:
        h.set_store_limit(3)
        with pytest.raises(pcb.PerCacheError) as e:
            h.prefill(G.specs_for(w.prompts, []))
        assert e.value.code == pcb.E_NOSPACE
        h.set_store_limit(4)
        h.prefill(G.specs_for(w.prompts, []))
        with pytest.raises(pcb.PerCacheError) as e:
            h.set_store_limit(2)
        assert e.value.code == pcb.E_NOSPACE and h.stats()["pages_used"] == 4
