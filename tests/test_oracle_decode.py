"""Pins of the decode oracle (CPU): a decode step is the last row of a prefill over one more token."""
import numpy as np
import pytest

from oracle import decode as dec
from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import workloads as wl
from tests.test_oracle_pins import _chunks, tiny_model


def test_decode_steps_equal_rows_of_a_dense_decoder():
    """Nothing cached, three layers, four decode steps: step j's output is row T + j of an ordinary causal
    decoder run over prompt + decoded tokens (an independent implementation: explicit mask, all rows)."""
    shape, weights, model = tiny_model(seed=51, n_layers=3)
    lens, nq, n_dec = [7, 12], 5, 4
    hs, qh = _chunks(shape, 51, lens, nq)
    toks = orc.bf16_bits_to_f64(wl.make_hidden(51, (3, 0), n_dec, shape.d_model))
    full, k_all, v_all = orc.dense_prefill(model, np.concatenate(hs + [qh, toks]))
    T = sum(lens) + nq
    store = orc.Store()
    res = orc.reuse_prefill(model, store, [orc.Prompt([100, 101], lens, hs, qh)], keep_ctx=True)[0]
    st = dec.begin_decode(res)
    assert st.n_tokens == T
    for j in range(n_dec):
        out = dec.decode_step(model, st, toks[j])
        assert st.n_tokens == T + j + 1
        assert np.allclose(out, full[T + j], atol=1e-9)
    # the grown context is the dense decoder's K (rotated) and V
    for l in range(3):
        assert np.array_equal(st.v_ctx[l], v_all[l])
        assert np.allclose(st.k_ctx[l], orc.rope(k_all[l], np.arange(T + n_dec), model.rope_theta), atol=1e-12)


@pytest.mark.parametrize("mask", [(1, 1, 1), (0, 1, 0), (1, 0, 1)])
def test_decode_after_reuse_prefill_equals_prefill_with_longer_query(mask):
    """With cached chunks (any mask, two layers): decoding token x after prefill(chunks, query) gives the last
    row of prefill(chunks, query + [x]) from the same store state."""
    shape, weights, model = tiny_model(seed=52, n_layers=2)
    lens, nq = [6, 9, 4], 3
    hs, qh = _chunks(shape, 52, lens, nq)
    tok = orc.bf16_bits_to_f64(wl.make_hidden(52, (3, 1), 2, shape.d_model))
    store = orc.Store()
    for i, n in enumerate(lens):
        if mask[i]:      # cached content made elsewhere: each chunk prefilled alone
            orc.reuse_prefill(model, store, [orc.Prompt([100 + i], [n], [hs[i]], np.zeros((0, shape.d_model)))])
    ids = [100, 101, 102]
    hid = [None if mask[i] else hs[i] for i in range(3)]
    res = orc.reuse_prefill(model, store, [orc.Prompt(ids, lens, hid, qh)], commit=False, keep_ctx=True)[0]
    st = dec.begin_decode(res)
    o1 = dec.decode_step(model, st, tok[0])
    o2 = dec.decode_step(model, st, tok[1])
    longer = orc.reuse_prefill(model, store, [orc.Prompt(ids, lens, hid, np.concatenate([qh, tok]))], commit=False)[0]
    assert np.allclose(o1, longer.out_hidden[-2], atol=1e-10)
    assert np.allclose(o2, longer.out_hidden[-1], atol=1e-10)


def test_decode_single_slot_context_closed_form():
    """One layer, a one-token prompt whose V dominates nothing: with zero attention weights on Wq the two
    visible slots get equal weight, so the attention output is the mean of the two V rows."""
    shape, weights, model = tiny_model(seed=53, n_layers=1, random_gains=False)
    weights[0]["wq"] = np.zeros_like(weights[0]["wq"])
    qh = orc.bf16_bits_to_f64(wl.make_hidden(53, (2, 0), 1, shape.d_model))
    tok = orc.bf16_bits_to_f64(wl.make_hidden(53, (3, 0), 1, shape.d_model))[0]
    res = orc.reuse_prefill(model, orc.Store(), [orc.Prompt([], [], [], qh)], keep_ctx=True)[0]
    st = dec.begin_decode(res)
    out = dec.decode_step(model, st, tok)
    v = st.v_ctx[0]                                            # [2, Hkv, hd]
    att = np.repeat(v.mean(axis=0), shape.n_q_heads // shape.n_kv_heads, axis=0).reshape(-1)
    x = tok + att @ model.w(0, "wo").T
    yn = orc.rmsnorm(x[None], model.w(0, "ffn_norm"), model.rms_eps)
    want = x + ((orc.silu(yn @ model.w(0, "w_gate").T) * (yn @ model.w(0, "w_up").T)) @ model.w(0, "w_down").T)[0]
    assert np.allclose(out, want, atol=1e-12)


def test_begin_decode_needs_the_context():
    shape, weights, model = tiny_model(seed=54, n_layers=1)
    qh = orc.bf16_bits_to_f64(wl.make_hidden(54, (2, 0), 2, shape.d_model))
    res = orc.reuse_prefill(model, orc.Store(), [orc.Prompt([], [], [], qh)])[0]
    with pytest.raises(ValueError):
        dec.begin_decode(res)
