"""Pins of the paper-faithful oracle (oracle/paper_mode.py) against the plain dense decoder, against itself served
from an empty cache, against hand-written chain lengths, and against the default mode's oracle.  CPU only."""
import numpy as np
import pytest

from oracle import paper_mode as pm
from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import workloads as wl
from tests import helpers as H
from tests.test_oracle_pins import _chunks, tiny_model


def _bf16_representable(x):
    return np.array_equal(orc.round_to_bf16(x), x)


def test_without_rounding_and_cache_it_is_the_dense_decoder():
    shape, weights, model = tiny_model(seed=51, n_layers=3)
    hs, qh = _chunks(shape, 51, [6, 9, 4], 5)
    full, _, _ = orc.dense_prefill(model, np.concatenate(hs + [qh]), round_kv=False)
    res = pm.paper_prefill(model, pm.PaperStore(), [pm.PaperPrompt([1, 2, 3], [6, 9, 4], hs, qh)], round_cache=False)[0]
    assert (res.n_matched, res.l_pre, res.l_total) == (0, 0, 24)
    assert np.allclose(res.out_hidden, full, atol=1e-10)


@pytest.mark.parametrize("n_prefix,drop", [(1, 0), (2, 0), (3, 0), (2, 3), (3, 4), (1, 6)])
def test_served_from_a_matched_chain_equals_served_from_an_empty_cache(n_prefix, drop):
    """Reuse is prefix-only, so every loaded tensor sits at the position it was computed at: the result must not
    depend on how much of the chain was loaded, nor on how many tail tokens were recomputed."""
    shape, weights, model = tiny_model(seed=52, n_layers=3)
    lens, nq = [6, 9, 4], 5
    hs, qh = _chunks(shape, 52, lens, nq)
    ids = [11, 12, 13]
    scratch = pm.paper_prefill(model, pm.PaperStore(), [pm.PaperPrompt(ids, lens, hs, qh)])[0]
    store = pm.PaperStore()
    pm.paper_prefill(model, store, [pm.PaperPrompt(ids[:n_prefix], lens[:n_prefix], hs[:n_prefix],
                                                   np.zeros((0, shape.d_model)))])
    assert sorted(store.qkv) == [tuple(ids[: i + 1]) for i in range(n_prefix)]
    res = pm.paper_prefill(model, store, [pm.PaperPrompt(ids, lens, hs, qh, tail_drop=drop)])[0]
    assert res.n_matched == n_prefix and res.l_pre == sum(lens[:n_prefix]) - drop and res.l_total == 24
    assert np.allclose(res.out_hidden, scratch.out_hidden, atol=1e-10)
    assert sorted(store.qkv) == [tuple(ids[: i + 1]) for i in range(3)]      # the missed nodes were added, the query not


def test_cached_tensors_are_bf16_in_context_slices_after_position_encoding():
    shape, weights, model = tiny_model(seed=53, n_layers=2)
    lens = [5, 7]
    hs, qh = _chunks(shape, 53, lens, 3)
    store = pm.PaperStore()
    pm.paper_prefill(model, store, [pm.PaperPrompt([1, 2], lens, hs, qh)])
    q2, k2, v2 = store.qkv[(1, 2)]
    assert q2.shape == (2, 7, shape.n_q_heads, shape.head_dim) and k2.shape == (2, 7, shape.n_kv_heads, shape.head_dim)
    assert _bf16_representable(q2) and _bf16_representable(k2) and _bf16_representable(v2)
    # layer 0 depends on the token alone: node (1, 2) holds chunk 2's projections rotated to positions 5..11
    xn = orc.rmsnorm(hs[1], model.w(0, "attn_norm"), model.rms_eps)
    k_want = orc.round_to_bf16(orc.rope((xn @ model.w(0, "wk").T).reshape(7, shape.n_kv_heads, shape.head_dim),
                                        np.arange(5, 12), model.rope_theta))
    q_want = orc.round_to_bf16(orc.rope((xn @ model.w(0, "wq").T).reshape(7, shape.n_q_heads, shape.head_dim),
                                        np.arange(5, 12), model.rope_theta))
    assert np.array_equal(k2[0], k_want) and np.array_equal(q2[0], q_want)
    # a different path to the same chunk is a different node
    assert not store.has((2,)) and store.has((1,)) and not store.has((2, 1))


def test_walk_stops_at_the_first_mismatch_and_length_is_checked():
    shape, weights, model = tiny_model(seed=54, n_layers=1)
    hs, qh = _chunks(shape, 54, [4, 4, 4], 2)
    store = pm.PaperStore()
    pm.paper_prefill(model, store, [pm.PaperPrompt([1, 2, 3], [4, 4, 4], hs, qh)])
    assert pm.match_chain(store, pm.PaperPrompt([1, 2, 3], [4, 4, 4], hs, qh)) == (3, 12)
    assert pm.match_chain(store, pm.PaperPrompt([1, 3, 2], [4, 4, 4], hs, qh)) == (1, 4)      # (1, 3) is not a node
    assert pm.match_chain(store, pm.PaperPrompt([2, 1], [4, 4], hs[:2], qh)) == (0, 0)
    assert pm.match_chain(store, pm.PaperPrompt([1, 2], [4, 4], hs[:2], qh, tail_drop=3)) == (2, 5)
    with pytest.raises(ValueError):
        pm.match_chain(store, pm.PaperPrompt([1, 2], [4, 5], hs[:2], qh))
    with pytest.raises(ValueError):
        pm.match_chain(store, pm.PaperPrompt([1, 2], [4, 4], hs[:2], qh, tail_drop=5))


def test_new_rows_agree_with_the_default_mode_in_prefix_matching():
    """Same matching rule, same new rows: the default mode (K/V only, rows of loaded chunks dropped for good) and the
    paper's (Q cached as well, all rows restored) give the same new rows when nothing is rounded, and differ by the
    placement of the bf16 rounding only (before or after position encoding; Q rounded or not) when it is."""
    shape, weights, model = tiny_model(seed=55, n_layers=3)
    lens, nq = [6, 9, 4], 5
    hs, qh = _chunks(shape, 55, lens, nq)
    ids = [1, 2, 3]
    for rounded, tol in ((False, 1e-9), (True, 5e-2)):
        ps, ds = pm.PaperStore(), orc.Store()
        pm.paper_prefill(model, ps, [pm.PaperPrompt(ids[:2], lens[:2], hs[:2], np.zeros((0, shape.d_model)))],
                         round_cache=rounded)
        orc.reuse_prefill(model, ds, [orc.Prompt(ids[:2], lens[:2], hs[:2], np.zeros((0, shape.d_model)))],
                          round_kv=rounded, match_prefix=True)
        a = pm.paper_prefill(model, ps, [pm.PaperPrompt(ids, lens, hs, qh)], round_cache=rounded)[0]
        b = orc.reuse_prefill(model, ds, [orc.Prompt(ids, lens, [None, None, hs[2]], qh)], round_kv=rounded,
                              match_prefix=True)[0]
        assert a.l_pre == 15 and b.layout.new_slots.tolist() == list(range(15, 24))
        assert np.max(np.abs(a.out_hidden[15:] - b.out_hidden)) < tol


def test_idempotence_and_batch_independence():
    shape, weights, model = tiny_model(seed=56, n_layers=2)
    hs, qh = _chunks(shape, 56, [8, 8], 4)
    store = pm.PaperStore()
    p1 = pm.PaperPrompt([1, 2], [8, 8], hs, qh)
    p2 = pm.PaperPrompt([1], [8], hs[:1], qh[:2])
    first = pm.paper_prefill(model, store, [p1, p2])
    assert [r.n_matched for r in first] == [0, 0]                # prompts of a batch do not see each other
    again = pm.paper_prefill(model, store, [p1, p2])
    assert [r.n_matched for r in again] == [2, 1]
    for a, b in zip(first, again):
        assert np.allclose(a.out_hidden, b.out_hidden, atol=1e-10)
