"""The paper-faithful mode (PERCACHE_FLAG_PAPER_MODE) through the C ABI against its oracle: prefix-tree matching,
cached Q, K and V, all L_total rows leaving every block, attention reading the pages through the page table."""
import numpy as np
import pytest

from oracle import paper_mode as pm
from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import percache as pcb
from paper_2601_11553_b200 import workloads as wl
from tests import gpu_helpers as G
from tests import helpers as H

pytestmark = pytest.mark.gpu
f64 = orc.bf16_bits_to_f64


def _handle(shape, weights, pool_pages, max_tokens, max_prompts=1, flags=0):
    return pcb.PerCache(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                        n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn, weights=weights,
                        pool_pages=pool_pages, max_prompt_tokens=max_tokens, max_batch_prompts=max_prompts,
                        flags=pcb.FLAG_PAPER_MODE | flags)


def test_sequence_of_queries_against_the_paper_mode_oracle():
    shape = wl.small_workload(seed=91, n_layers=3, chunk_lens=[16], n_query=1, hit_idx=[]).shape
    weights = wl.make_weights(shape, 91, random_gains=True)
    model = H.oracle_model(shape, weights)
    lens = {1: 128, 5: 96, 7: 32, 9: 160, 12: 64}
    hid = {c: wl.chunk_hidden_for(91, c, n, shape.d_model) for c, n in lens.items()}
    # (chunk list, tail drop, expected hit mask)
    queries = [([1, 5, 7], 0, [0, 0, 0]), ([1, 5, 9], 0, [1, 1, 0]), ([1, 5, 9, 12], 32, [1, 1, 1, 0]),
               ([5, 1], 0, [0, 0]), ([1, 5, 7], 16, [1, 1, 1]), ([1, 9], 128, [1, 0])]
    store = pm.PaperStore()
    with _handle(shape, weights, 256, 600) as h:
        for qi, (ids, drop, want_mask) in enumerate(queries):
            qh = wl.make_hidden(91, (2, qi), 21 + 7 * qi, shape.d_model)
            want = pm.paper_prefill(model, store, [pm.PaperPrompt(ids, [lens[c] for c in ids], [f64(hid[c]) for c in ids],
                                                                  f64(qh), tail_drop=drop)])[0]
            got = h.prefill([pcb.PromptSpec(ids, [lens[c] for c in ids], [hid[c] for c in ids], qh, match_prefix=True,
                                            tail_drop=drop)])[0]
            assert got.hit_mask.tolist() == want_mask and int(sum(want_mask)) == want.n_matched, qi
            assert got.n_total == want.l_total and got.n_new == want.l_total - want.l_pre, qi
            assert got.out_hidden.shape[0] == want.l_total                     # every row comes back
            c = G.compare_hidden(got.out_hidden, want.out_hidden)
            assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (qi, c)
            # and against the plain dense decoder over the whole prompt (the mode equals it up to the bf16 cache)
            full, _, _ = orc.dense_prefill(model, np.concatenate([f64(hid[c]) for c in ids] + [f64(qh)]), round_kv=False)
            c = G.compare_hidden(got.out_hidden, full)
            assert c["max_abs"] <= 2 * G.TOL_MAX_ABS and c["mean_abs"] <= 2 * G.TOL_MEAN_ABS, (qi, c)
        # the nodes hold Q, K (both rotated) and V as the oracle's store does
        for path in [(1,), (1, 5), (1, 5, 9), (1, 5, 9, 12), (5, 1)]:
            key = pcb.path_key(list(path))
            assert h.has_chunk(key) == lens[path[-1]]
            q_want, k_want, v_want = store.qkv[path]
            k_bits, v_bits = h.get_chunk_kv(key)
            q_bits = h.get_chunk_q(key)
            for bits, wv in ((q_bits, q_want), (k_bits, k_want), (v_bits, v_want)):
                g = f64(bits).reshape(wv.shape)
                step = 2.0 ** (np.floor(np.log2(np.maximum(np.maximum(np.abs(wv), np.abs(g)), 2.0 ** -20))) - 7)
                # block 0 depends on the token alone: fp16 operand rounding moves a sum by ~1e-3, then the bf16
                # rounding may fall one step apart; deeper blocks inherit the hidden-state tolerance
                assert np.all(np.abs(g[0] - wv[0]) <= 1.001 * step[0] + 2e-3)
                assert np.max(np.abs(g - wv)) <= G.TOL_MAX_ABS
                assert np.mean(np.abs(f64(bits).reshape(wv.shape) - wv)) <= G.TOL_MEAN_ABS
        assert h.has_chunk(pcb.path_key([9])) is None and h.has_chunk(1) is None
        pages_before = h.stats()["pages_free"]
        # scratch pages of the query rows were returned: a second identical call leaves the free count unchanged
        ids = [1, 5, 9, 12]
        qh = wl.make_hidden(91, (2, 77), 40, shape.d_model)
        a = h.prefill([pcb.PromptSpec(ids, [lens[c] for c in ids], [hid[c] for c in ids], qh, match_prefix=True)])[0]
        b = h.prefill([pcb.PromptSpec(ids, [lens[c] for c in ids], [hid[c] for c in ids], qh, match_prefix=True)])[0]
        assert h.stats()["pages_free"] == pages_before and a.hit_mask.tolist() == [1, 1, 1, 1]
        # same pages, same arithmetic (up to the order of the atomic additions of a K-split residual GEMM)
        assert np.max(np.abs(a.out_hidden - b.out_hidden)) < 1e-4


def test_batch_and_refusals():
    shape = wl.small_workload(seed=92, n_layers=2, chunk_lens=[16], n_query=1, hit_idx=[]).shape
    weights = wl.make_weights(shape, 92, random_gains=True)
    model = H.oracle_model(shape, weights)
    lens = {1: 64, 2: 144, 3: 32}
    hid = {c: wl.chunk_hidden_for(92, c, n, shape.d_model) for c, n in lens.items()}
    q0 = wl.make_hidden(92, (2, 0), 130, shape.d_model)
    q1 = wl.make_hidden(92, (2, 1), 5, shape.d_model)
    store = pm.PaperStore()
    with _handle(shape, weights, 128, 400, max_prompts=2) as h:
        for rnd in range(2):     # first all misses (both prompts compute node (1,), prompt 0 keeps it), then hits
            prompts = [([1, 2], q0), ([1, 3], q1)]
            want = pm.paper_prefill(model, store, [pm.PaperPrompt(ids, [lens[c] for c in ids], [f64(hid[c]) for c in ids],
                                                                  f64(q)) for ids, q in prompts])
            got = h.prefill([pcb.PromptSpec(ids, [lens[c] for c in ids], [hid[c] for c in ids], q, match_prefix=True)
                             for ids, q in prompts])
            for g, wnt in zip(got, want):
                assert g.hit_mask.tolist() == ([0, 0] if rnd == 0 else [1, 1])
                c = G.compare_hidden(g.out_hidden, wnt.out_hidden)
                assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, (rnd, c)
        assert h.stats()["pages_used"] == (64 + 144 + 32) // 16

        def code(fn):
            with pytest.raises(pcb.PerCacheError) as e:
                fn()
            return e.value.code
        odd = wl.chunk_hidden_for(92, 8, 40, shape.d_model)
        assert code(lambda: h.prefill([pcb.PromptSpec([8], [40], [odd], q1, match_prefix=True)])) == pcb.E_INVAL
        assert code(lambda: h.prefill([pcb.PromptSpec([1], [64], [hid[1]], q1)])) == pcb.E_INVAL          # id matching
        assert code(lambda: h.prefill([pcb.PromptSpec([1], [64], [None], q1, match_prefix=True)])) == pcb.E_MISS_NO_INPUT
        assert code(lambda: h.prefill([pcb.PromptSpec([1], [64], [hid[1]], q1, match_prefix=True, tail_drop=8)])) == pcb.E_INVAL
        kz = np.zeros((2, 16, shape.kv_dim), np.uint16)
        assert code(lambda: h.put_chunk_kv(99, kz, kz)) == pcb.E_INVAL
        assert code(lambda: h.decode(np.zeros((2, shape.d_model), np.uint16))) == pcb.E_INVAL


def test_config1_shape_prefix_hits_two_layers():
    """The 28-layer workload's shape and prompt (8 x 256 + 64 tokens) at two layers, first four chunks cached as a
    chain: 17 tiles of rows, attention units cut along the context, CTA-pair GEMMs on all 2112 rows."""
    shape = wl.ModelShape(n_layers=2, **wl.SHAPE_A)
    weights = wl.make_weights(shape, 1, random_gains=True)
    model = H.oracle_model(shape, weights)
    ids = list(range(8))
    hid = [wl.chunk_hidden_for(1, c, 256, shape.d_model) for c in ids]
    qh = wl.make_hidden(1, (2, 0), 64, shape.d_model)
    store = pm.PaperStore()
    with _handle(shape, weights, 8 * 16 + 16, 2112) as h:
        pm.paper_prefill(model, store, [pm.PaperPrompt(ids[:4], [256] * 4, [f64(x) for x in hid[:4]],
                                                       np.zeros((0, shape.d_model)))])
        h.prefill([pcb.PromptSpec(ids[:4], [256] * 4, hid[:4], None, 0, match_prefix=True)])
        want = pm.paper_prefill(model, store, [pm.PaperPrompt(ids, [256] * 8, [f64(x) for x in hid], f64(qh))])[0]
        got = h.prefill([pcb.PromptSpec(ids, [256] * 8, hid, qh, match_prefix=True)])[0]
        assert got.hit_mask.tolist() == [1, 1, 1, 1, 0, 0, 0, 0] and got.n_new == 1088 and got.n_total == 2112
        c = G.compare_hidden(got.out_hidden, want.out_hidden)
        print("paper mode, config-1 shape, 2 layers:", c, h.stats()["device_us"])
        assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, c
