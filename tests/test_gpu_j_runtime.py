"""Runtime behaviour around the kernels: the fp16 operand range, a bounded wait that runs out, handles on more
than one device, and what a failed call leaves behind when eviction is on."""
import numpy as np
import pytest
import torch

from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import percache as pcb
from paper_2601_11553_b200 import workloads as wl
from tests import gpu_helpers as G
from tests import helpers as H

pytestmark = pytest.mark.gpu

F16_MAX = 65504.0


def _scaled(bits: np.ndarray, factor: float) -> np.ndarray:
    return wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(bits) * np.float32(factor))


def test_large_but_representable_activations_still_match_the_oracle():
    """Operands are fp16: values up to 65504 are carried.  Hidden states of magnitude ~1e3 (the norm removes the
    scale) and FFN weights scaled so that silu(gate) * up reaches ~1e4 must still agree with the oracle, relative
    to the size of the outputs."""
    w = wl.small_workload(seed=81, n_layers=1, chunk_lens=[64, 40], n_query=24, hit_idx=[0])
    weights = wl.make_weights(w.shape, w.seed, random_gains=True)
    for lw in weights:
        lw["w_gate"] = _scaled(lw["w_gate"], 40.0)
        lw["w_up"] = _scaled(lw["w_up"], 400.0)
    p = w.prompts[0]
    p.chunk_hidden = [_scaled(hh, 1000.0) for hh in p.chunk_hidden]
    p.query_hidden = _scaled(p.query_hidden, 1000.0)
    model = H.oracle_model(w.shape, weights)
    # cached chunk: K/V of the same (scaled) inputs, so its values are ordinary
    store = orc.Store()
    orc.reuse_prefill(model, store, [orc.Prompt([p.chunk_ids[0]], [p.chunk_len[0]],
                                                [orc.bf16_bits_to_f64(p.chunk_hidden[0])], np.zeros((0, w.shape.d_model)))])
    want = orc.reuse_prefill(model, store, [H.oracle_prompt(p, [0])], commit=False)[0]
    with G.make_handle(w.shape, weights, w.prompts) as h:
        G.push_store(h, store, w.cached_ids)
        got = h.prefill(G.specs_for(w.prompts, w.cached_ids))[0]
    scale = float(np.max(np.abs(want.out_hidden)))
    act_peak = scale          # for the record: outputs are of the order of the FFN product times |w_down|
    err = np.abs(got.out_hidden.astype(np.float64) - want.out_hidden)
    print("output scale", scale, "max err", err.max(), "mean err", err.mean(), act_peak)
    assert np.all(np.isfinite(got.out_hidden))
    assert err.max() <= 3e-2 * max(1.0, scale / 10.0) and err.mean() <= 3e-3 * max(1.0, scale / 10.0)


def test_values_beyond_the_fp16_range_saturate_and_stay_finite():
    """The documented behaviour beyond +-65504: the store keeps bf16 values as given, every fp16 operand formed from
    them clips to +-65504, and no infinity or NaN appears downstream."""
    w = wl.small_workload(seed=82, n_layers=2, chunk_lens=[32, 48], n_query=16, hit_idx=[0])
    weights = wl.make_weights(w.shape, w.seed)
    for lw in weights:
        lw["w_up"] = _scaled(lw["w_up"], 3.0e5)          # silu(gate) * up far beyond 65504
    p = w.prompts[0]
    L, n, kvd = w.shape.n_layers, p.chunk_len[0], w.shape.kv_dim
    rng = np.random.default_rng(82)
    big = (rng.standard_normal((L, n, kvd)) * 3.0e5).astype(np.float32)       # cached K/V far beyond the fp16 range
    kb, vb = wl.f32_to_bf16_bits(big), wl.f32_to_bf16_bits(big[::-1].copy())
    with G.make_handle(w.shape, weights, w.prompts) as h:
        h.put_chunk_kv(p.chunk_ids[0], kb, vb)
        k_back, v_back = h.get_chunk_kv(p.chunk_ids[0])
        assert np.array_equal(k_back, kb) and np.array_equal(v_back, vb)       # the store is bf16: nothing clipped
        got = h.prefill(G.specs_for(w.prompts, w.cached_ids))[0]
        assert np.all(np.isfinite(got.out_hidden))
        k_ctx, v_ctx = h.read_ctx(0, 0, got.n_total)
        assert np.all(np.isfinite(k_ctx)) and np.all(np.isfinite(v_ctx))
        want_v = np.clip(wl.bf16_bits_to_f32(vb[0]), -F16_MAX, F16_MAX).astype(np.float16)
        assert np.array_equal(v_ctx[:n], want_v)                               # gathered V: clipped, else exact
        assert np.max(np.abs(k_ctx[:n].astype(np.float32))) == F16_MAX         # rotated K reaches the clip value
        # the store now also holds the missed chunk; its pages must be finite bf16
        k2, _ = h.get_chunk_kv(p.chunk_ids[1])
        assert np.all(np.isfinite(wl.bf16_bits_to_f32(k2)))


def test_bounded_wait_runs_out_and_the_device_stays_usable():
    rc, code, waited = pcb.debug_wait_probe(limit_us=1000)
    assert rc == pcb.E_DEVICE_TIMEOUT and code == 901
    assert 1.0e6 <= waited[0] < 50.0e6            # the first waiter gave up after its own limit (1 ms)...
    assert waited[1] < 100.0e6                    # ...and the second long before its own (1 s): it saw the error word
    a = (np.random.default_rng(5).standard_normal((200, 256)) * 0.5).astype(np.float16)
    b = (np.random.default_rng(6).standard_normal((256, 256)) * 0.5).astype(np.float16)
    c = pcb.debug_gemm(a, b)
    assert np.max(np.abs(c - a.astype(np.float64) @ b.astype(np.float64).T)) < 1e-2
    rc2, code2, _ = pcb.debug_wait_probe(limit_us=200)
    assert rc2 == pcb.E_DEVICE_TIMEOUT and code2 == 901


def _one_prefill(device: int, seed: int):
    w = wl.small_workload(seed=seed, n_layers=1, chunk_lens=[64, 64], n_query=8, hit_idx=[])
    weights = wl.make_weights(w.shape, w.seed, random_gains=True)
    model = H.oracle_model(w.shape, weights)
    want = orc.reuse_prefill(model, orc.Store(), [H.oracle_prompt(w.prompts[0])])[0]
    p = w.prompts[0]
    h = pcb.PerCache(n_layers=1, d_model=w.shape.d_model, n_q_heads=w.shape.n_q_heads, n_kv_heads=w.shape.n_kv_heads,
                     head_dim=128, d_ffn=w.shape.d_ffn, weights=weights, pool_pages=64, max_prompt_tokens=p.n_total,
                     device=device)
    return h, w, want


def test_two_handles_on_one_device_and_handles_on_two_devices():
    """Kernel attributes are per device: a second handle (same device, and another device where one is visible) must
    launch its kernels with the attributes set there too."""
    devices = [0, 0] + ([1] if torch.cuda.device_count() > 1 else [])
    handles = [_one_prefill(dev, 83 + i) for i, dev in enumerate(devices)]
    try:
        for h, w, want in handles + handles[::-1]:
            got = h.prefill(G.specs_for(w.prompts, [c for c in w.prompts[0].chunk_ids if h.has_chunk(c) is not None]))[0]
            if got.n_new == want.out_hidden.shape[0]:
                c = G.compare_hidden(got.out_hidden, want.out_hidden)
                assert c["max_abs"] <= G.TOL_MAX_ABS and c["mean_abs"] <= G.TOL_MEAN_ABS, c
            else:      # second pass: the chunks are stored now, only the query rows are computed
                assert got.n_new == w.prompts[0].n_query and got.hit_mask.tolist() == [1, 1]
    finally:
        for h, _, _ in handles:
            h.close()


def test_failed_call_with_eviction_on_leaves_the_store_as_it_was():
    """With least-frequently-used eviction on, the victims of a call are only dropped when its device work starts: a
    call that is refused on the host after they were chosen changes nothing."""
    shape = wl.small_workload(seed=84, n_layers=1, chunk_lens=[16], n_query=1, hit_idx=[]).shape
    weights = wl.make_weights(shape, 84)
    mk = lambda cid, n: wl.chunk_hidden_for(84, cid, n, shape.d_model)
    q = wl.make_hidden(84, (2, 0), 4, shape.d_model)
    h = pcb.PerCache(n_layers=1, d_model=shape.d_model, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                     head_dim=128, d_ffn=shape.d_ffn, weights=weights, pool_pages=4, max_prompt_tokens=200,
                     flags=pcb.FLAG_EVICT_LFU)
    with h:
        h.prefill([pcb.PromptSpec([1, 2], [32, 32], [mk(1, 32), mk(2, 32)], q)])        # the store is full: 4 pages
        before = (h.chunk_info(1), h.chunk_info(2), h.stats()["pages_free"])
        small = np.empty(8, dtype=np.float32)
        h.capture_layers(small)           # a capture buffer that is too small: refused after the victims were chosen
        with pytest.raises(pcb.PerCacheError) as e:
            h.prefill([pcb.PromptSpec([3], [48], [mk(3, 48)], q)])
        h.capture_layers(None)
        assert e.value.code == pcb.E_CAPACITY
        assert (h.chunk_info(1), h.chunk_info(2), h.stats()["pages_free"]) == before and h.has_chunk(3) is None
        # the same call without the obstacle evicts both and stores chunk 3
        h.prefill([pcb.PromptSpec([3], [48], [mk(3, 48)], q)])
        assert h.stats()["evictions"] == 2 and h.has_chunk(1) is None and h.has_chunk(2) is None and h.has_chunk(3) == 48
        assert h.stats()["pages_free"] == 1
