"""CPU oracle for reuse-prefill.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition the CUDA library is checked against.  It
is imported by the tests, by the smoke check and by the benchmark's CPU-baseline
leg, and by nothing else: the product never routes through it, and it shares no
code with the CUDA path.

What it computes (paper Section 3.2.2 "QKV Cache Reuse" and Appendix B.1
"Inference implementation details"):

  * a prompt is an ordered list of knowledge chunks followed by the user's query
    tokens (Section 3, system overview; Section 3.2.1);
  * tensors of chunks found in the cache are loaded and concatenated in order, the
    length already covered is recorded so positions can be calibrated
    (Section 3.2.2; Appendix B.1, L_pre / L_total);
  * within every transformer block the rows that correspond to loaded tensors are
    dropped from the attention input, projection and position encoding run on the
    remaining rows only, with the position counter offset so every row gets its
    true position in the full sequence (Appendix B.1, RoPE paragraph);
  * computed and loaded tensors are concatenated on the sequence axis and "the
    subsequent operations proceed normally" (Appendix B.1);
  * tensors collected during prefill are sliced per chunk on the sequence
    dimension and saved, one entry per chunk (Section 3.2.1, cache slicer).

Readings taken where the paper is silent or this library deliberately differs
(each is listed in the design notes): only K and V are cached; K is cached before
rotation and rotated to the slot's position when loaded (for a prefix hit this is
the paper's scheme exactly); any chunk of the list may hit, not only a prefix;
only the new rows (missed chunks + query) continue through the block; cached K/V
is bf16, so freshly computed K/V is rounded to bf16 before use; RoPE pairs element
i with i + head_dim/2; Q head h reads KV head h // (Hq/Hkv); pre-norm residual
blocks with RMSNorm and a SwiGLU FFN, no biases, no final norm.

Arithmetic is float64 throughout (numpy); the single rounding is K/V -> bf16.

Parity pins (tests/test_oracle_*.py): a Llama decoder from an independent library
in float64 (dense case), brute-force attention in Python loops, RoPE identities,
closed forms, causality, the single-layer "reuse == full prefill" invariant, the
prefix-reuse invariant at any depth, and idempotence.  Unpinned: non-prefix hits
at more than one layer have no definition outside this algorithm ("parity
unpinned" for that case; the single-layer and prefix invariants bracket it).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------- #
# number formats
# --------------------------------------------------------------------------- #
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 to the nearest bf16 value (8 significant bits, ties to even), as float64.

    The cache format is bf16, so this defines what a stored K/V element is.  Done
    directly from float64 (no intermediate float32 step): write x = m * 2^e with
    0.5 <= |m| < 1, keep 8 bits of m.  Magnitudes below the bf16 normal range keep
    the fixed spacing 2^-133 of bf16 subnormals.
    """
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)
    e = np.maximum(e, -125)                      # subnormal spacing below 2^-126
    q = np.rint(np.ldexp(x, 8 - e))              # np.rint rounds half to even
    return np.ldexp(q, e - 8)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Bit patterns of values that already are bf16-representable."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    return (f.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# --------------------------------------------------------------------------- #
# the pieces of a block
# --------------------------------------------------------------------------- #
def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x * rsqrt(mean(x^2) + eps) * gain over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope_angles(positions: np.ndarray, head_dim: int, theta: float) -> np.ndarray:
    """angle[p, i] = p * theta^(-2i/head_dim), i in [0, head_dim/2)."""
    half = head_dim // 2
    inv_freq = np.power(float(theta), -2.0 * np.arange(half, dtype=np.float64) / head_dim)
    return np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]


def rope(x: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotate x [n, heads, head_dim] to `positions` [n]; element i is paired with i + head_dim/2.

    The position is the row's index in the full sequence, not its index among the
    computed rows (Appendix B.1: the position counter is offset by L_pre).
    """
    n, h, hd = x.shape
    half = hd // 2
    ang = rope_angles(positions, hd, theta)
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def attention_rows(q: np.ndarray, q_pos: np.ndarray, k: np.ndarray, v: np.ndarray) -> np.ndarray:
    """Causal grouped-query attention of some rows against a whole context.

    q [m, Hq, hd] (rotated) at positions q_pos [m]; k (rotated), v [T, Hkv, hd] for
    slots 0..T-1 whose position equals the slot index.  Row r sees slots t <= q_pos[r].
    Returns [m, Hq*hd].
    """
    m, hq, hd = q.shape
    T, hkv, _ = k.shape
    group = hq // hkv
    scale = 1.0 / np.sqrt(float(hd))
    visible = np.arange(T)[None, :] <= np.asarray(q_pos)[:, None]          # [m, T]
    out = np.empty((m, hq, hd), dtype=np.float64)
    for h in range(hq):
        g = h // group
        s = (q[:, h, :] @ k[:, g, :].T) * scale                            # [m, T]
        s = np.where(visible, s, -np.inf)
        s = s - np.max(s, axis=1, keepdims=True)
        p = np.exp(s)
        p = p / np.sum(p, axis=1, keepdims=True)
        out[:, h, :] = p @ v[:, g, :]
    return out.reshape(m, hq * hd)


# --------------------------------------------------------------------------- #
# model, store, prompt
# --------------------------------------------------------------------------- #
@dataclass
class Model:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    rope_theta: float
    rms_eps: float
    # per layer: dict name -> bf16 bits [out, in] (projections) or [d] (norm gains)
    layers: List[Dict[str, np.ndarray]] = field(default_factory=list)

    def w(self, layer: int, name: str) -> np.ndarray:
        return bf16_bits_to_f64(self.layers[layer][name])


@dataclass
class Prompt:
    chunk_ids: Sequence[int]
    chunk_len: Sequence[int]
    chunk_hidden: Sequence[Optional[np.ndarray]]      # float64 [len, d] or None (expected hit)
    query_hidden: np.ndarray                          # float64 [n_query, d]
    # Prefix matching only (Appendix B, "Tokenization Inconsistency", second measure): the tensors of the last
    # `tail_drop` tokens of the final matched node are discarded and those tokens are computed from their inputs.
    tail_drop: int = 0


@dataclass
class Layout:
    """Integer description of one assembled prompt (the part that must match bit for bit)."""
    n_total: int
    hit_mask: np.ndarray          # uint8 [n_chunks]
    slot_chunk: np.ndarray        # int32 [T]: index into the prompt's chunk list, n_chunks for query tokens
    slot_offset: np.ndarray       # int32 [T]: token index inside its chunk (or inside the query)
    slot_is_new: np.ndarray       # uint8 [T]
    new_slots: np.ndarray         # int32 [n_new]: slots of new rows, ascending (= their positions)


class MissNoInput(Exception):
    pass


class LengthMismatch(Exception):
    pass


class Store:
    """chunk id -> (K, V), each float64 [n_layers, n_tokens, Hkv, hd] holding bf16 values, K unrotated."""

    def __init__(self):
        self.kv: Dict[int, Tuple[np.ndarray, np.ndarray]] = {}

    def has(self, cid: int) -> bool:
        return cid in self.kv

    def put(self, cid: int, k: np.ndarray, v: np.ndarray) -> None:
        if cid in self.kv:
            raise KeyError(f"chunk {cid} already stored")
        self.kv[cid] = (np.array(k, dtype=np.float64), np.array(v, dtype=np.float64))

    def drop(self, cid: int) -> None:
        del self.kv[cid]


def store_keys(prompt: Prompt, match_prefix: bool) -> List:
    """Key of every chunk of the prompt in the store.

    By id: the chunk id.  By prefix (paper Section 3.2.1: each node of the cache tree is a chunk and each path
    a chunk list retrieved by a query): the tuple of ids from the first chunk of the list down to this one.
    """
    if not match_prefix:
        return list(prompt.chunk_ids)
    return [tuple(prompt.chunk_ids[: i + 1]) for i in range(len(prompt.chunk_ids))]


def assemble_layout(store: Store, prompt: Prompt, match_prefix: bool = False) -> Layout:
    """Slots 0..T-1 are the chunks in the given order, then the query; position(t) = t.

    A chunk hits when its key is stored (with the same length); every other chunk,
    and every query token, is a new row (Section 3.2.2: only the part not covered by
    loaded tensors is retained and computed).  With match_prefix the walk of Section
    3.2.2 is taken: first chunk, then the second as its child, ... and it stops at the
    first mismatch, after which every chunk is new.
    """
    n_chunks = len(prompt.chunk_ids)
    hit = np.zeros(n_chunks, dtype=np.uint8)
    slot_chunk: List[int] = []
    slot_off: List[int] = []
    is_new: List[int] = []
    keys = store_keys(prompt, match_prefix)
    walking = True
    for i, (cid, n) in enumerate(zip(keys, prompt.chunk_len)):
        if store.has(cid) and store.kv[cid][0].shape[1] != n:
            raise LengthMismatch(f"chunk {cid}: stored {store.kv[cid][0].shape[1]} tokens, prompt says {n}")
        if store.has(cid) and (walking or not match_prefix):
            hit[i] = 1
        else:
            walking = False
            if prompt.chunk_hidden is None or i >= len(prompt.chunk_hidden) or prompt.chunk_hidden[i] is None:
                raise MissNoInput(f"chunk {cid} missed and no hidden states were given")
    # the final matched node keeps only its first chunk_len - tail_drop tokens (prefix matching only)
    drop = int(getattr(prompt, "tail_drop", 0) or 0)
    last_hit = int(np.nonzero(hit)[0][-1]) if hit.any() else -1
    if drop:
        if not match_prefix or drop < 0:
            raise ValueError("tail_drop needs prefix matching and a non-negative count")
        if last_hit >= 0:
            if drop > prompt.chunk_len[last_hit]:
                raise ValueError("tail_drop exceeds the length of the final matched chunk")
            if prompt.chunk_hidden is None or last_hit >= len(prompt.chunk_hidden) or prompt.chunk_hidden[last_hit] is None:
                raise MissNoInput("tail_drop needs the hidden states of the final matched chunk")
    for i, n in enumerate(prompt.chunk_len):
        reuse_len = n - drop if (i == last_hit and drop) else n
        for o in range(n):
            slot_chunk.append(i)
            slot_off.append(o)
            is_new.append(0 if (hit[i] and o < reuse_len) else 1)
    nq = 0 if prompt.query_hidden is None else prompt.query_hidden.shape[0]
    for o in range(nq):
        slot_chunk.append(n_chunks)
        slot_off.append(o)
        is_new.append(1)
    is_new_a = np.asarray(is_new, dtype=np.uint8)
    return Layout(
        n_total=len(slot_chunk), hit_mask=hit,
        slot_chunk=np.asarray(slot_chunk, dtype=np.int32), slot_offset=np.asarray(slot_off, dtype=np.int32),
        slot_is_new=is_new_a, new_slots=np.nonzero(is_new_a)[0].astype(np.int32))


@dataclass
class PromptResult:
    layout: Layout
    out_hidden: np.ndarray                      # float64 [n_new, d]: final residual of the new rows
    # assembled context of every layer (rotated K, V) — kept only when asked for
    k_ctx: Optional[List[np.ndarray]] = None
    v_ctx: Optional[List[np.ndarray]] = None


def reuse_prefill(model: Model, store: Store, prompts: Sequence[Prompt], commit: bool = True,
                  keep_ctx: bool = False, round_kv: bool = True, match_prefix: bool = False) -> List[PromptResult]:
    """Prefill a batch of prompts, taking the K/V of stored chunks from the store.

    Hits are decided against the store as it is when the call starts; the prompts of
    a batch do not see each other.  After the call every missed chunk is stored
    (its K/V as computed inside this prompt, sliced on the sequence axis), query
    tokens are not.  If two prompts miss the same chunk the first one's slices are kept.
    """
    layouts = [assemble_layout(store, p, match_prefix) for p in prompts]     # raises before anything changes
    results: List[PromptResult] = []
    pending: List[Tuple[int, np.ndarray, np.ndarray]] = []
    hkv, hd, hq = model.n_kv_heads, model.head_dim, model.n_q_heads
    for prompt, lay in zip(prompts, layouts):
        T = lay.n_total
        n_chunks = len(prompt.chunk_ids)
        new = lay.new_slots
        m = new.shape[0]
        # layer input of the new rows, in slot order
        x = np.empty((m, model.d_model), dtype=np.float64)
        for r, t in enumerate(new):
            c, o = int(lay.slot_chunk[t]), int(lay.slot_offset[t])
            x[r] = prompt.query_hidden[o] if c == n_chunks else prompt.chunk_hidden[c][o]
        pos_all = np.arange(T)
        k_pre_layers: List[np.ndarray] = []
        v_layers: List[np.ndarray] = []
        kc_keep: List[np.ndarray] = []
        vc_keep: List[np.ndarray] = []
        for l in range(model.n_layers):
            xn = rmsnorm(x, model.w(l, "attn_norm"), model.rms_eps)
            q = (xn @ model.w(l, "wq").T).reshape(m, hq, hd)
            k = (xn @ model.w(l, "wk").T).reshape(m, hkv, hd)
            v = (xn @ model.w(l, "wv").T).reshape(m, hkv, hd)
            if round_kv:
                k, v = round_to_bf16(k), round_to_bf16(v)          # what the cache would hold
            # unrotated K and V of every slot: loaded for hits, just computed for new rows
            k_pre = np.empty((T, hkv, hd), dtype=np.float64)
            v_all = np.empty((T, hkv, hd), dtype=np.float64)
            k_pre[new] = k
            v_all[new] = v
            start = 0
            for i, (cid, n) in enumerate(zip(store_keys(prompt, match_prefix), prompt.chunk_len)):
                if lay.hit_mask[i]:                                 # load and place in order
                    ck, cv = store.kv[cid]
                    reused = lay.slot_is_new[start:start + n] == 0      # all of the chunk unless its tail is dropped
                    k_pre[start:start + n][reused] = ck[l][reused]
                    v_all[start:start + n][reused] = cv[l][reused]
                start += n
            k_rot = rope(k_pre, pos_all, model.rope_theta)          # every slot at its own position
            q_rot = rope(q, new, model.rope_theta)
            att = attention_rows(q_rot, new, k_rot, v_all)
            x = x + att @ model.w(l, "wo").T
            yn = rmsnorm(x, model.w(l, "ffn_norm"), model.rms_eps)
            act = silu(yn @ model.w(l, "w_gate").T) * (yn @ model.w(l, "w_up").T)
            x = x + act @ model.w(l, "w_down").T
            k_pre_layers.append(k_pre)
            v_layers.append(v_all)
            if keep_ctx:
                kc_keep.append(k_rot)
                vc_keep.append(v_all)
        # slice the collected K/V of missed chunks on the sequence axis, one slice per chunk
        start = 0
        for i, (cid, n) in enumerate(zip(store_keys(prompt, match_prefix), prompt.chunk_len)):
            if not lay.hit_mask[i]:
                ks = np.stack([kl[start:start + n] for kl in k_pre_layers])
                vs = np.stack([vl[start:start + n] for vl in v_layers])
                pending.append((cid, ks, vs))
            start += n
        results.append(PromptResult(lay, x, kc_keep if keep_ctx else None, vc_keep if keep_ctx else None))
    if commit:
        for cid, ks, vs in pending:
            if not store.has(cid):
                store.put(cid, ks, vs)
    return results


# --------------------------------------------------------------------------- #
# one block, some rows: the unit of a teacher-forced check
# --------------------------------------------------------------------------- #
def block_rows(model: Model, layer: int, x: np.ndarray, new_slots: np.ndarray, n_total: int,
               hit_segments: Sequence[Tuple[int, np.ndarray, np.ndarray]], rows: np.ndarray,
               round_kv: bool = True) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """One transformer block of reuse-prefill for one prompt, with the block's output formed for some rows only.

    The same steps as the loop body of reuse_prefill (Appendix B.1: projection and position encoding on the rows
    that are not covered by loaded tensors, computed and loaded tensors concatenated on the sequence axis, the rest
    of the block as usual), arranged so that a full-size case can be checked block by block: the K and V of a
    block depend on the block's input for *every* new row, but attention, output projection and FFN are row-wise,
    so they are evaluated for the chosen rows alone.

    x            float64 [m, d]: the block's input for all m new rows of the prompt, in slot order
    new_slots    int [m]: their slots (= positions), ascending
    n_total      context length T of the prompt
    hit_segments [(first slot, K [n, Hkv, hd], V [n, Hkv, hd])]: this layer's stored (unrotated, bf16-valued)
                 tensors of the chunks that hit, each with the slot its first token occupies
    rows         indices into the m new rows
    Returns (block output of the chosen rows [len(rows), d], unrotated K of all new rows, V of all new rows).
    """
    hq, hkv, hd = model.n_q_heads, model.n_kv_heads, model.head_dim
    new = np.asarray(new_slots)
    rows = np.asarray(rows)
    m = x.shape[0]
    xn = rmsnorm(x, model.w(layer, "attn_norm"), model.rms_eps)
    k = (xn @ model.w(layer, "wk").T).reshape(m, hkv, hd)
    v = (xn @ model.w(layer, "wv").T).reshape(m, hkv, hd)
    if round_kv:
        k, v = round_to_bf16(k), round_to_bf16(v)
    k_pre = np.zeros((n_total, hkv, hd), dtype=np.float64)
    v_all = np.zeros((n_total, hkv, hd), dtype=np.float64)
    k_pre[new] = k
    v_all[new] = v
    for start, ck, cv in hit_segments:
        k_pre[start:start + ck.shape[0]] = ck
        v_all[start:start + cv.shape[0]] = cv
    pos_r = new[rows]
    t_hi = int(pos_r.max()) + 1 if rows.size else 0          # no chosen row sees a slot beyond this one
    k_rot = rope(k_pre[:t_hi], np.arange(t_hi), model.rope_theta)
    q = (xn[rows] @ model.w(layer, "wq").T).reshape(rows.size, hq, hd)
    q_rot = rope(q, pos_r, model.rope_theta)
    att = attention_rows(q_rot, pos_r, k_rot, v_all[:t_hi])
    xr = x[rows] + att @ model.w(layer, "wo").T
    yn = rmsnorm(xr, model.w(layer, "ffn_norm"), model.rms_eps)
    act = silu(yn @ model.w(layer, "w_gate").T) * (yn @ model.w(layer, "w_up").T)
    xr = xr + act @ model.w(layer, "w_down").T
    return xr, k, v


# --------------------------------------------------------------------------- #
# the plain definition without any cache: every row goes through every block
# --------------------------------------------------------------------------- #
def dense_prefill(model: Model, hidden: np.ndarray, round_kv: bool = True):
    """Ordinary causal decoder prefill of hidden [T, d] (the "naive inference without cache").

    Returns (final residual [T, d], K [L, T, Hkv, hd] unrotated, V [L, T, Hkv, hd]).
    Written separately from reuse_prefill: explicit lower-triangular mask, all rows.
    """
    T = hidden.shape[0]
    hq, hkv, hd = model.n_q_heads, model.n_kv_heads, model.head_dim
    rep = hq // hkv
    pos = np.arange(T)
    tril = np.tril(np.ones((T, T), dtype=bool))
    x = np.array(hidden, dtype=np.float64)
    ks, vs = [], []
    for l in range(model.n_layers):
        h = rmsnorm(x, model.w(l, "attn_norm"), model.rms_eps)
        q = (h @ model.w(l, "wq").T).reshape(T, hq, hd)
        k = (h @ model.w(l, "wk").T).reshape(T, hkv, hd)
        v = (h @ model.w(l, "wv").T).reshape(T, hkv, hd)
        if round_kv:
            k, v = round_to_bf16(k), round_to_bf16(v)
        ks.append(k)
        vs.append(v)
        qr = rope(q, pos, model.rope_theta)
        kr = np.repeat(rope(k, pos, model.rope_theta), rep, axis=1)     # [T, Hq, hd]
        vr = np.repeat(v, rep, axis=1)
        o = np.empty((T, hq, hd), dtype=np.float64)
        for hh in range(hq):
            s = qr[:, hh] @ kr[:, hh].T / np.sqrt(float(hd))
            s = np.where(tril, s, -np.inf)
            e = np.exp(s - s.max(axis=1, keepdims=True))
            o[:, hh] = (e / e.sum(axis=1, keepdims=True)) @ vr[:, hh]
        x = x + o.reshape(T, hq * hd) @ model.w(l, "wo").T
        h2 = rmsnorm(x, model.w(l, "ffn_norm"), model.rms_eps)
        x = x + (silu(h2 @ model.w(l, "w_gate").T) * (h2 @ model.w(l, "w_up").T)) @ model.w(l, "w_down").T
    return x, np.stack(ks), np.stack(vs)
