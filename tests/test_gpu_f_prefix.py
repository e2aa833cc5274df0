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
