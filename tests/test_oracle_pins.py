"""Pins of the CPU oracle against things other than itself.

Each test fixes the oracle to a closed form, an identity, a brute-force loop, a
hand-written expectation, or an independent library (a Llama decoder in float64),
so that a dropped term, a wrong sign or index, or a transposed operand anywhere in
it fails at least one of them.  No GPU is involved.
"""
import math
import os

import numpy as np
import pytest

from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import workloads as wl
from tests import helpers as H

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def tiny_shape(n_layers=2, d=64, hq=4, hkv=2, hd=16, f=96):
    return wl.ModelShape(n_layers=n_layers, d_model=d, n_q_heads=hq, n_kv_heads=hkv, head_dim=hd, d_ffn=f)


def tiny_model(seed=11, std=0.08, random_gains=True, **kw):
    shape = tiny_shape(**kw)
    weights = wl.make_weights(shape, seed, std=std)
    if random_gains:                       # gains != 1 so a dropped gain is caught
        for l, w in enumerate(weights):
            rng = np.random.default_rng([seed, 99, l])
            w["attn_norm"] = wl.f32_to_bf16_bits(1.0 + 0.3 * rng.standard_normal(shape.d_model).astype(np.float32))
            w["ffn_norm"] = wl.f32_to_bf16_bits(1.0 + 0.3 * rng.standard_normal(shape.d_model).astype(np.float32))
    return shape, weights, H.oracle_model(shape, weights)


# --------------------------------------------------------------------------- #
# number format
# --------------------------------------------------------------------------- #
def test_bf16_rounding_hand_values():
    cases = []
    with open(os.path.join(GOLDEN, "bf16_rounding.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                a, b = line.split()
                cases.append((float.fromhex(a), float.fromhex(b)))
    assert len(cases) >= 8
    for x, want in cases:
        assert orc.round_to_bf16(np.array([x]))[0] == want, (x, want)
        assert orc.round_to_bf16(np.array([-x]))[0] == -want


def test_bf16_rounding_matches_library_cast():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(5)
    x32 = (rng.standard_normal(200000) * np.exp(rng.uniform(-20, 20, 200000))).astype(np.float32)
    want = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    got = orc.round_to_bf16(x32.astype(np.float64))
    assert np.array_equal(got, want)
    # and the bit helpers round-trip
    bits = orc.f64_to_bf16_bits(got)
    assert np.array_equal(orc.bf16_bits_to_f64(bits), got)
    assert np.array_equal(bits, wl.f32_to_bf16_bits(x32))


def test_bf16_rounding_is_direct_from_float64():
    # 1 + 2^-8 + 2^-40 lies just above the tie: must round up even though a float32
    # intermediate (which drops the 2^-40) would make it a tie and round down to even.
    x = 1.0 + 2.0 ** -8 + 2.0 ** -40
    assert orc.round_to_bf16(np.array([x]))[0] == 1.0 + 2.0 ** -7


# --------------------------------------------------------------------------- #
# textbook pieces
# --------------------------------------------------------------------------- #
def test_rmsnorm_closed_forms():
    g = np.linspace(0.5, 1.5, 8)
    x = np.full((3, 8), 2.0)
    want = 2.0 / math.sqrt(4.0 + 1e-6) * g
    assert np.allclose(orc.rmsnorm(x, g, 1e-6), want[None, :], rtol=0, atol=1e-15)
    # hand loop on random input
    rng = np.random.default_rng(0)
    x = rng.standard_normal((2, 8))
    for r in range(2):
        ms = sum(v * v for v in x[r]) / 8.0
        for j in range(8):
            assert abs(orc.rmsnorm(x, g, 1e-5)[r, j] - x[r, j] / math.sqrt(ms + 1e-5) * g[j]) < 1e-14


def test_silu_values():
    assert orc.silu(np.array([0.0]))[0] == 0.0
    for v in (-3.0, -0.5, 0.7, 4.0):
        assert abs(orc.silu(np.array([v]))[0] - v / (1.0 + math.exp(-v))) < 1e-15
    # large |x|: silu(x) -> x, silu(-x) -> 0
    assert abs(orc.silu(np.array([40.0]))[0] - 40.0) < 1e-12
    assert abs(orc.silu(np.array([-40.0]))[0]) < 1e-12


# --------------------------------------------------------------------------- #
# RoPE
# --------------------------------------------------------------------------- #
def test_rope_angle_definition_by_hand():
    hd, theta = 8, 1.0e6
    ang = orc.rope_angles(np.array([0, 1, 7, 33023]), hd, theta)
    for pi, p in enumerate([0, 1, 7, 33023]):
        for i in range(hd // 2):
            assert abs(ang[pi, i] - p * theta ** (-2.0 * i / hd)) <= 1e-12 * max(1.0, p)


def test_rope_pairing_half_split_by_hand():
    hd, theta = 8, 1.0e6
    x = np.zeros((1, 1, hd))
    x[0, 0, 1] = 1.0                                   # element 1 pairs with element 1 + hd/2 = 5
    p = 3
    y = orc.rope(x, np.array([p]), theta)[0, 0]
    a = p * theta ** (-2.0 * 1 / hd)
    want = np.zeros(hd)
    want[1], want[5] = math.cos(a), math.sin(a)
    assert np.allclose(y, want, atol=1e-15)
    x[:] = 0.0
    x[0, 0, 5] = 1.0
    y = orc.rope(x, np.array([p]), theta)[0, 0]
    want[:] = 0.0
    want[1], want[5] = -math.sin(a), math.cos(a)
    assert np.allclose(y, want, atol=1e-15)


def test_rope_identities():
    rng = np.random.default_rng(1)
    hd, theta = 128, 1.0e6
    x = rng.standard_normal((5, 3, hd))
    # R(0) = I exactly
    assert np.array_equal(orc.rope(x, np.zeros(5, dtype=np.int64), theta), x)
    pa = np.array([3, 10, 999, 20000, 33023])
    pb = np.array([7, 1, 24, 13000, 1])
    ya = orc.rope(x, pa, theta)
    # pairwise norm preserved
    half = hd // 2
    n0 = x[..., :half] ** 2 + x[..., half:] ** 2
    n1 = ya[..., :half] ** 2 + ya[..., half:] ** 2
    assert np.allclose(n0, n1, rtol=1e-12)
    # R(a) R(b) = R(a + b)
    assert np.allclose(orc.rope(ya, pb, theta), orc.rope(x, pa + pb, theta), atol=1e-9)
    # <R(m) q, R(n) k> depends on m - n only
    q = rng.standard_normal((5, 3, hd))
    k = rng.standard_normal((5, 3, hd))
    d0 = np.sum(orc.rope(q, pa, theta) * orc.rope(k, pb, theta), axis=-1)
    d1 = np.sum(orc.rope(q, pa + 500, theta) * orc.rope(k, pb + 500, theta), axis=-1)
    assert np.allclose(d0, d1, atol=1e-8)


# --------------------------------------------------------------------------- #
# attention
# --------------------------------------------------------------------------- #
def brute_attention(q, q_pos, k, v):
    m, hq, hd = q.shape
    T, hkv, _ = k.shape
    grp = hq // hkv
    out = np.zeros((m, hq, hd))
    for r in range(m):
        for h in range(hq):
            g = h // grp
            sc = []
            for t in range(T):
                if t <= q_pos[r]:
                    sc.append(sum(q[r, h, e] * k[t, g, e] for e in range(hd)) / math.sqrt(hd))
            mx = max(sc)
            ex = [math.exp(s - mx) for s in sc]
            z = sum(ex)
            for t in range(len(sc)):
                for e in range(hd):
                    out[r, h, e] += ex[t] / z * v[t, g, e]
    return out.reshape(m, hq * hd)


def test_attention_vs_brute_force():
    rng = np.random.default_rng(2)
    T, hq, hkv, hd = 13, 4, 2, 8
    k = rng.standard_normal((T, hkv, hd))
    v = rng.standard_normal((T, hkv, hd))
    q_pos = np.array([0, 4, 5, 9, 12])
    q = rng.standard_normal((len(q_pos), hq, hd)) * 2.0
    got = orc.attention_rows(q, q_pos, k, v)
    assert np.allclose(got, brute_attention(q, q_pos, k, v), atol=1e-12)


def test_attention_closed_forms():
    rng = np.random.default_rng(3)
    T, hq, hkv, hd = 9, 4, 2, 8
    k = rng.standard_normal((T, hkv, hd))
    v = rng.standard_normal((T, hkv, hd))
    q_pos = np.array([0, 3, 8])
    q = np.zeros((3, hq, hd))
    out = orc.attention_rows(q, q_pos, k, v).reshape(3, hq, hd)
    for r, p in enumerate(q_pos):                # zero query: mean of V over the visible slots
        for h in range(hq):
            assert np.allclose(out[r, h], v[: p + 1, h // 2].mean(axis=0), atol=1e-14)
    # a row at position 0 sees one slot: output is V[0] whatever q is
    q = rng.standard_normal((1, hq, hd))
    out = orc.attention_rows(q, np.array([0]), k, v).reshape(hq, hd)
    for h in range(hq):
        assert np.allclose(out[h], v[0, h // 2], atol=1e-15)
    # GQA mapping is by contiguous groups: heads 0,1 -> kv 0; heads 2,3 -> kv 1
    q = np.zeros((1, hq, hd))
    v2 = np.zeros((T, hkv, hd))
    v2[:, 1, :] = 1.0
    out = orc.attention_rows(q, np.array([T - 1]), k, v2).reshape(hq, hd)
    assert np.all(out[:2] == 0.0) and np.allclose(out[2:], 1.0)


# --------------------------------------------------------------------------- #
# layout assembly (integer part) against a hand-written expectation
# --------------------------------------------------------------------------- #
def test_layout_by_hand():
    store = orc.Store()
    z = lambda n: np.zeros((1, n, 1, 2))
    store.put(7, z(3), z(3))
    store.put(9, z(2), z(2))
    d = 4
    pr = orc.Prompt(chunk_ids=[7, 5, 9], chunk_len=[3, 2, 2],
                    chunk_hidden=[None, np.zeros((2, d)), None], query_hidden=np.zeros((2, d)))
    lay = orc.assemble_layout(store, pr)
    assert lay.n_total == 9
    assert lay.hit_mask.tolist() == [1, 0, 1]
    assert lay.slot_chunk.tolist() == [0, 0, 0, 1, 1, 2, 2, 3, 3]
    assert lay.slot_offset.tolist() == [0, 1, 2, 0, 1, 0, 1, 0, 1]
    assert lay.slot_is_new.tolist() == [0, 0, 0, 1, 1, 0, 0, 1, 1]
    assert lay.new_slots.tolist() == [3, 4, 7, 8]
    # length disagreement and a miss without input are errors
    with pytest.raises(orc.LengthMismatch):
        orc.assemble_layout(store, orc.Prompt([7], [4], [None], np.zeros((1, d))))
    with pytest.raises(orc.MissNoInput):
        orc.assemble_layout(store, orc.Prompt([8], [4], [None], np.zeros((1, d))))


# --------------------------------------------------------------------------- #
# dense case against an independent library implementation
# --------------------------------------------------------------------------- #
def hf_llama_hidden(shape, weights, hidden):
    torch = pytest.importorskip("torch")
    tr = pytest.importorskip("transformers")
    cfg = tr.LlamaConfig(hidden_size=shape.d_model, intermediate_size=shape.d_ffn,
                         num_hidden_layers=shape.n_layers + 1, num_attention_heads=shape.n_q_heads,
                         num_key_value_heads=shape.n_kv_heads, head_dim=shape.head_dim,
                         rms_norm_eps=shape.rms_eps, rope_theta=shape.rope_theta, attention_bias=False,
                         mlp_bias=False, vocab_size=8, max_position_embeddings=4096)
    m = tr.LlamaModel(cfg).double().eval()
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj",
             "wo": "self_attn.o_proj", "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj",
             "w_down": "mlp.down_proj", "attn_norm": "input_layernorm", "ffn_norm": "post_attention_layernorm"}
    with torch.no_grad():
        for l in range(shape.n_layers):
            sd = dict(m.layers[l].named_parameters())
            for k, n in names.items():
                sd[n + ".weight"].copy_(torch.from_numpy(orc.bf16_bits_to_f64(weights[l][k])))
        o = m(inputs_embeds=torch.from_numpy(hidden)[None], output_hidden_states=True)
    # hidden_states[L] is the input of the extra block = un-normed output of block L-1
    return o.hidden_states[shape.n_layers][0].numpy()


@pytest.mark.parametrize("hd", [16, 128])
def test_dense_prefill_matches_library_llama(hd):
    shape, weights, model = tiny_model(seed=21, n_layers=3, hd=hd, d=64, f=96)
    rng = np.random.default_rng(4)
    hidden = orc.bf16_bits_to_f64(wl.f32_to_bf16_bits(rng.standard_normal((23, shape.d_model)).astype(np.float32)))
    want = hf_llama_hidden(shape, weights, hidden)
    got, _, _ = orc.dense_prefill(model, hidden, round_kv=False)
    # the library takes cos/sin in float32, hence 1e-5 rather than 1e-12
    assert np.max(np.abs(got - want)) < 2e-5 * max(1.0, np.max(np.abs(want)))


def test_reuse_prefill_all_new_matches_library_llama():
    shape, weights, model = tiny_model(seed=22, n_layers=2)
    rng = np.random.default_rng(6)
    mk = lambda n: orc.bf16_bits_to_f64(wl.f32_to_bf16_bits(rng.standard_normal((n, shape.d_model)).astype(np.float32)))
    hs = [mk(5), mk(7), mk(4)]
    pr = orc.Prompt([1, 2], [5, 7], hs[:2], hs[2])
    res = orc.reuse_prefill(model, orc.Store(), [pr], round_kv=False)[0]
    want = hf_llama_hidden(shape, weights, np.concatenate(hs))
    assert res.out_hidden.shape == want.shape
    assert np.max(np.abs(res.out_hidden - want)) < 2e-5 * max(1.0, np.max(np.abs(want)))


# --------------------------------------------------------------------------- #
# invariants of the reuse path
# --------------------------------------------------------------------------- #
def _chunks(shape, seed, lens, nq):
    hs = [orc.bf16_bits_to_f64(wl.chunk_hidden_for(seed, 100 + i, n, shape.d_model)) for i, n in enumerate(lens)]
    qh = orc.bf16_bits_to_f64(wl.make_hidden(seed, (2, 0), nq, shape.d_model))
    return hs, qh


@pytest.mark.parametrize("mask", [(1, 1, 1, 1), (0, 1, 0, 1), (1, 0, 1, 0), (0, 0, 1, 1), (0, 0, 0, 0)])
def test_single_layer_reuse_equals_full_prefill_any_mask(mask):
    """One layer, cached K/V made from the same inputs: reuse == full prefill on the new rows."""
    shape, weights, model = tiny_model(seed=31, n_layers=1)
    lens, nq = [5, 16, 3, 9], 6
    hs, qh = _chunks(shape, 31, lens, nq)
    full, k_all, v_all = orc.dense_prefill(model, np.concatenate(hs + [qh]))
    store = orc.Store()
    # K/V of layer 0 depends on the token alone, so per-chunk K/V computed anywhere is the same
    for i, n in enumerate(lens):
        if mask[i]:
            _, kc, vc = orc.dense_prefill(model, hs[i])
            store.put(100 + i, kc, vc)
    pr = orc.Prompt([100 + i for i in range(4)], lens, [None if mask[i] else hs[i] for i in range(4)], qh)
    res = orc.reuse_prefill(model, store, [pr], keep_ctx=True)[0]
    assert res.layout.hit_mask.tolist() == list(mask)
    assert np.allclose(res.out_hidden, full[res.layout.new_slots], atol=1e-10)
    # the assembled context is the full prefill's K (rotated) and V
    assert np.array_equal(res.v_ctx[0], v_all[0])
    assert np.allclose(res.k_ctx[0], orc.rope(k_all[0], np.arange(sum(lens) + nq), model.rope_theta), atol=1e-12)


@pytest.mark.parametrize("n_prefix", [1, 2, 3])
def test_prefix_reuse_equals_full_prefill_any_depth(n_prefix):
    """Hits form a prefix whose K/V came from a prefill of exactly that prefix (the paper's case)."""
    shape, weights, model = tiny_model(seed=32, n_layers=3)
    lens, nq = [6, 17, 4], 5
    hs, qh = _chunks(shape, 32, lens, nq)
    full, _, _ = orc.dense_prefill(model, np.concatenate(hs + [qh]))
    # populate: prefill the prefix chunks together (no query); this stores in-context slices
    store = orc.Store()
    ids = [100, 101, 102]
    orc.reuse_prefill(model, store, [orc.Prompt(ids[:n_prefix], lens[:n_prefix], hs[:n_prefix],
                                                np.zeros((0, shape.d_model)))])
    assert sorted(store.kv) == ids[:n_prefix]
    pr = orc.Prompt(ids, lens, [None] * n_prefix + hs[n_prefix:], qh)
    res = orc.reuse_prefill(model, store, [pr])[0]
    assert res.layout.hit_mask.tolist() == [1] * n_prefix + [0] * (3 - n_prefix)
    assert np.allclose(res.out_hidden, full[res.layout.new_slots], atol=1e-9)
    # misses were committed, the query was not
    assert sorted(store.kv) == ids


def test_commit_holds_in_context_slices_and_idempotence():
    shape, weights, model = tiny_model(seed=33, n_layers=2)
    lens, nq = [4, 7], 3
    hs, qh = _chunks(shape, 33, lens, nq)
    _, k_all, v_all = orc.dense_prefill(model, np.concatenate(hs + [qh]))
    store = orc.Store()
    pr = orc.Prompt([100, 101], lens, hs, qh)
    r1 = orc.reuse_prefill(model, store, [pr])[0]
    assert np.allclose(store.kv[100][0], k_all[:, 0:4], atol=1e-12)
    assert np.allclose(store.kv[101][0], k_all[:, 4:11], atol=1e-12)
    assert np.allclose(store.kv[101][1], v_all[:, 4:11], atol=1e-12)
    # second call: all hits, query rows reproduce the first call's query rows
    r2 = orc.reuse_prefill(model, store, [orc.Prompt([100, 101], lens, [None, None], qh)])[0]
    assert r2.layout.hit_mask.tolist() == [1, 1]
    assert r2.out_hidden.shape[0] == nq
    assert np.allclose(r2.out_hidden, r1.out_hidden[-nq:], atol=1e-10)


def test_failed_call_leaves_store_unchanged_and_commit_off():
    shape, weights, model = tiny_model(seed=34, n_layers=1)
    hs, qh = _chunks(shape, 34, [4, 5], 2)
    store = orc.Store()
    with pytest.raises(orc.MissNoInput):
        orc.reuse_prefill(model, store, [orc.Prompt([100], [4], [hs[0]], qh),
                                         orc.Prompt([101], [5], [None], qh)])
    assert not store.kv
    orc.reuse_prefill(model, store, [orc.Prompt([100], [4], [hs[0]], qh)], commit=False)
    assert not store.kv


def test_batch_prompts_are_independent_and_first_miss_wins():
    shape, weights, model = tiny_model(seed=35, n_layers=2)
    hs, qh = _chunks(shape, 35, [4, 5], 2)
    p0 = orc.Prompt([100, 101], [4, 5], hs, qh)
    p1 = orc.Prompt([101], [5], [hs[1]], qh)
    s = orc.Store()
    both = orc.reuse_prefill(model, s, [p0, p1])
    alone0 = orc.reuse_prefill(model, orc.Store(), [p0])[0]
    alone1 = orc.reuse_prefill(model, orc.Store(), [p1])[0]
    assert np.array_equal(both[0].out_hidden, alone0.out_hidden)
    assert np.array_equal(both[1].out_hidden, alone1.out_hidden)
    s0 = orc.Store()
    orc.reuse_prefill(model, s0, [p0])
    assert np.array_equal(s.kv[101][0], s0.kv[101][0])      # chunk 101 as computed inside prompt 0


def test_causality():
    shape, weights, model = tiny_model(seed=36, n_layers=2)
    hs, qh = _chunks(shape, 36, [5, 6], 4)
    base = orc.reuse_prefill(model, orc.Store(), [orc.Prompt([100, 101], [5, 6], hs, qh)])[0].out_hidden
    qh2 = qh.copy()
    qh2[2] += 1.0                                            # slot 5 + 6 + 2 = 13
    pert = orc.reuse_prefill(model, orc.Store(), [orc.Prompt([100, 101], [5, 6], hs, qh2)])[0].out_hidden
    assert np.array_equal(pert[:13], base[:13])
    assert np.max(np.abs(pert[13:] - base[13:])) > 1e-3


def test_position_of_new_rows_is_their_slot_not_their_row_index():
    """A hit in front must move the new rows' positions (the offset by L_pre of Appendix B.1)."""
    shape, weights, model = tiny_model(seed=37, n_layers=1)
    hs, qh = _chunks(shape, 37, [8], 3)
    _, kc, vc = orc.dense_prefill(model, hs[0])
    store = orc.Store()
    store.put(100, kc, vc)
    with_hit = orc.reuse_prefill(model, store, [orc.Prompt([100], [8], [None], qh)], keep_ctx=True)[0]
    # rotated K of the query slots must equal K rotated at positions 8, 9, 10
    xn = orc.rmsnorm(qh, model.w(0, "attn_norm"), model.rms_eps)
    k = orc.round_to_bf16((xn @ model.w(0, "wk").T).reshape(3, shape.n_kv_heads, shape.head_dim))
    assert np.allclose(with_hit.k_ctx[0][8:], orc.rope(k, np.array([8, 9, 10]), model.rope_theta), atol=1e-12)
    assert not np.allclose(with_hit.k_ctx[0][8:], orc.rope(k, np.array([0, 1, 2]), model.rope_theta), atol=1e-3)


# --------------------------------------------------------------------------- #
# prefix-tree matching (the paper's walk): reuse equals full prefill, call after call
# --------------------------------------------------------------------------- #
def test_prefix_tree_walk_hand_cases():
    store = orc.Store()
    z = lambda n: np.zeros((1, n, 1, 2))
    store.put((7,), z(3), z(3))
    store.put((7, 9), z(2), z(2))
    store.put((5,), z(2), z(2))
    store.put((8, 9, 4), z(1), z(1))            # a node whose ancestors are gone
    d = 4
    hid = lambda n: np.zeros((n, d))
    # 7 -> 9 matches two levels, then 5 is not a child of (7, 9): computed, although (5,) exists as a root
    lay = orc.assemble_layout(store, orc.Prompt([7, 9, 5], [3, 2, 2], [None, None, hid(2)], hid(1)), match_prefix=True)
    assert lay.hit_mask.tolist() == [1, 1, 0]
    # 9 is not a root: nothing matches, the walk stops at once
    lay = orc.assemble_layout(store, orc.Prompt([9, 7], [2, 3], [hid(2), hid(3)], hid(1)), match_prefix=True)
    assert lay.hit_mask.tolist() == [0, 0]
    # ancestors missing: the stored descendant is not used
    lay = orc.assemble_layout(store, orc.Prompt([8, 9, 4], [1, 2, 1], [hid(1), hid(2), hid(1)], hid(1)), match_prefix=True)
    assert lay.hit_mask.tolist() == [0, 0, 0]
    # by id, any stored chunk matches anywhere
    store.put(9, z(2), z(2))
    lay = orc.assemble_layout(store, orc.Prompt([3, 9], [1, 2], [hid(1), None], hid(1)))
    assert lay.hit_mask.tolist() == [0, 1]


def test_prefix_tree_reuse_equals_full_prefill_over_a_sequence_of_queries():
    shape, weights, model = tiny_model(seed=38, n_layers=3)
    lens = {1: 6, 5: 9, 7: 4, 9: 11, 12: 5}
    hs = {c: orc.bf16_bits_to_f64(wl.chunk_hidden_for(38, c, n, shape.d_model)) for c, n in lens.items()}
    store = orc.Store()
    queries = [([1, 5, 7], [0, 0, 0]), ([1, 5, 9], [1, 1, 0]), ([1, 5, 9, 12], [1, 1, 1, 0]), ([5, 1], [0, 0]),
               ([1, 5, 7], [1, 1, 1]), ([1, 9], [1, 0])]
    for qi, (ids, want_mask) in enumerate(queries):
        qh = orc.bf16_bits_to_f64(wl.make_hidden(38, (2, qi), 3, shape.d_model))
        pr = orc.Prompt(ids, [lens[c] for c in ids], [hs[c] for c in ids], qh)
        res = orc.reuse_prefill(model, store, [pr], match_prefix=True)[0]
        assert res.layout.hit_mask.tolist() == want_mask, (qi, res.layout.hit_mask)
        full, _, _ = orc.dense_prefill(model, np.concatenate([hs[c] for c in ids] + [qh]))
        assert np.allclose(res.out_hidden, full[res.layout.new_slots], atol=1e-9), qi
    assert (1, 5, 9, 12) in store.kv and (5, 1) in store.kv and (1,) in store.kv and 1 not in store.kv


# --------------------------------------------------------------------------- #
# the block-by-block form used for teacher-forced checks at full size
# --------------------------------------------------------------------------- #
def _hit_segments(store, prompt, layout, layer):
    segs, start = [], 0
    for i, (cid, n) in enumerate(zip(prompt.chunk_ids, prompt.chunk_len)):
        if layout.hit_mask[i]:
            segs.append((start, store.kv[cid][0][layer], store.kv[cid][1][layer]))
        start += n
    return segs


@pytest.mark.parametrize("mask", [(1, 0, 1), (0, 0, 0), (0, 1, 1)])
def test_block_rows_chained_over_layers_is_reuse_prefill(mask):
    """block_rows fed its own outputs, all rows chosen, walks the same path as reuse_prefill (itself pinned to an
    independent decoder); with a subset of rows it returns exactly those rows; and with prefix hits the chain ends
    at plain full prefill."""
    shape, weights, model = tiny_model(seed=35, n_layers=3)
    lens, nq = [7, 16, 5], 6
    hs, qh = _chunks(shape, 35, lens, nq)
    ids = [100, 101, 102]
    store = orc.Store()
    for i in range(3):            # cached content computed in some other context: each chunk alone
        if mask[i]:
            orc.reuse_prefill(model, store, [orc.Prompt([ids[i]], [lens[i]], [hs[i]], np.zeros((0, shape.d_model)))])
    pr = orc.Prompt(ids, lens, [None if mask[i] else hs[i] for i in range(3)], qh)
    want = orc.reuse_prefill(model, store, [pr], commit=False, keep_ctx=True)[0]
    lay = want.layout
    m = lay.new_slots.shape[0]
    x = np.concatenate([hs[i] for i in range(3) if not mask[i]] + [qh])
    some = np.array([0, m // 2, m - 1])
    for l in range(3):
        out_all, k_new, v_new = orc.block_rows(model, l, x, lay.new_slots, lay.n_total,
                                               _hit_segments(store, pr, lay, l), np.arange(m))
        out_some, _, _ = orc.block_rows(model, l, x, lay.new_slots, lay.n_total, _hit_segments(store, pr, lay, l), some)
        assert np.allclose(out_some, out_all[some], atol=1e-12)
        # the new rows' V is what reuse_prefill put into the assembled context at those slots
        assert np.array_equal(v_new, want.v_ctx[l][lay.new_slots])
        assert np.allclose(orc.rope(k_new, lay.new_slots, model.rope_theta), want.k_ctx[l][lay.new_slots], atol=1e-12)
        x = out_all
    assert np.allclose(x, want.out_hidden, atol=1e-10)


def test_block_rows_with_prefix_hits_ends_at_full_prefill():
    shape, weights, model = tiny_model(seed=36, n_layers=2)
    lens, nq = [9, 12], 4
    hs, qh = _chunks(shape, 36, lens, nq)
    full, k_all, v_all = orc.dense_prefill(model, np.concatenate(hs + [qh]))
    new = np.arange(lens[0], sum(lens) + nq)
    x = np.concatenate([hs[1], qh])
    for l in range(2):
        x, _, _ = orc.block_rows(model, l, x, new, sum(lens) + nq, [(0, k_all[l][:lens[0]], v_all[l][:lens[0]])],
                                 np.arange(new.shape[0]))
    assert np.allclose(x, full[new], atol=1e-9)


def test_block_rows_hit_segment_placement_matters():
    """A segment placed one slot off, or K and V swapped, must change the result (the check is not vacuous)."""
    shape, weights, model = tiny_model(seed=37, n_layers=1)
    hs, qh = _chunks(shape, 37, [8, 8], 3)
    _, kc, vc = orc.dense_prefill(model, hs[0])
    new = np.arange(8, 19)
    x = np.concatenate([hs[1], qh])
    rows = np.arange(11)
    good, _, _ = orc.block_rows(model, 0, x, new, 19, [(0, kc[0], vc[0])], rows)
    swapped, _, _ = orc.block_rows(model, 0, x, new, 19, [(0, vc[0], kc[0])], rows)
    assert np.max(np.abs(good - swapped)) > 1e-3
    rolled, _, _ = orc.block_rows(model, 0, x, new, 19, [(0, np.roll(kc[0], 1, axis=0), np.roll(vc[0], 1, axis=0))], rows)
    assert np.max(np.abs(good - rolled)) > 1e-4


@pytest.mark.parametrize("drop", [0, 1, 5, 17])
def test_prefix_reuse_with_the_tail_of_the_last_matched_chunk_recomputed(drop):
    """Appendix B, tokenisation paragraph, second measure: the last few tokens of the final matched node are computed
    from their inputs instead of being loaded.  Layout by hand; and since the recomputed rows see the same prefix,
    the result still is plain full prefill."""
    shape, weights, model = tiny_model(seed=38, n_layers=2)
    lens, nq = [6, 17, 4], 5
    hs, qh = _chunks(shape, 38, lens, nq)
    full, _, _ = orc.dense_prefill(model, np.concatenate(hs + [qh]))
    store = orc.Store()
    orc.reuse_prefill(model, store, [orc.Prompt([100, 101], lens[:2], hs[:2], np.zeros((0, shape.d_model)))],
                      match_prefix=True)
    pr = orc.Prompt([100, 101, 102], lens, [None, hs[1], hs[2]], qh, tail_drop=drop)
    res = orc.reuse_prefill(model, store, [pr], match_prefix=True, commit=False)[0]
    lay = res.layout
    assert lay.hit_mask.tolist() == [1, 1, 0]
    l_pre = 6 + 17 - drop                                   # L_pre of Appendix B.1
    assert lay.slot_is_new.tolist() == [0] * l_pre + [1] * (32 - l_pre)
    assert lay.new_slots.tolist() == list(range(l_pre, 32))
    assert lay.slot_chunk.tolist() == [0] * 6 + [1] * 17 + [2] * 4 + [3] * 5
    assert np.allclose(res.out_hidden, full[l_pre:], atol=1e-9)


def test_tail_drop_is_refused_outside_prefix_matching_and_without_inputs():
    shape, weights, model = tiny_model(seed=39, n_layers=1)
    hs, qh = _chunks(shape, 39, [8, 8], 2)
    store = orc.Store()
    orc.reuse_prefill(model, store, [orc.Prompt([1, 2], [8, 8], hs, np.zeros((0, shape.d_model)))], match_prefix=True)
    with pytest.raises(orc.MissNoInput):
        orc.reuse_prefill(model, store, [orc.Prompt([1, 2], [8, 8], [None, None], qh, tail_drop=3)], match_prefix=True)
    with pytest.raises(ValueError):
        orc.reuse_prefill(model, store, [orc.Prompt([1, 2], [8, 8], hs, qh, tail_drop=9)], match_prefix=True)
    st2 = orc.Store()
    orc.reuse_prefill(model, st2, [orc.Prompt([1, 2], [8, 8], hs, np.zeros((0, shape.d_model)))])
    with pytest.raises(ValueError):
        orc.reuse_prefill(model, st2, [orc.Prompt([1, 2], [8, 8], hs, qh, tail_drop=3)])
