"""CPU oracle for the paper-faithful form of QKV-cache reuse.  TEST INFRASTRUCTURE ONLY.

Slow, plain numpy float64; imported by tests and by the benchmark's CPU legs, never by the product, and it shares
no code with the CUDA path.  It states the scheme exactly as the paper gives it, where oracle/reuse_prefill.py
states the library's default reading (K and V only, any-position hits, only new rows continue):

  * the cache is a tree whose nodes are chunks and whose paths are the chunk lists of earlier queries
    (Section 3.2.1); a new query's list is matched from its first chunk downwards until the first mismatch
    (Section 3.2.2);
  * a node holds the chunk's Q, K and V slices of every block, collected from the attention module during a
    prefill (Section 3.2.1 "collect and save the QKV tensors"; Section 5.3 shows all three projections skipped),
    K and Q as they are used by attention, i.e. after position encoding -- valid because a node is only ever reused
    at the position it was computed at (prefix matching);
  * at query time (Appendix B.1) the whole prompt is embedded (L_total rows); in every block the first L_pre rows
    of the block's input are cropped away, the QKV projection runs on the remaining L_total - L_pre rows, position
    encoding is applied with the position counter offset by L_pre, the loaded tensors are concatenated in front,
    which restores the sequence length to L_total, and the rest of the block proceeds as usual on all L_total
    rows; the output has L_total rows;
  * for a matched chain the tensors of the last few tokens of its final node may be discarded and recomputed
    (Appendix B, "Tokenization Inconsistency", second measure): `tail_drop`.

Readings: the store is bf16, so Q (rotated), K (rotated) and V are rounded to bf16 before attention uses them,
for loaded and for freshly computed rows alike (what the cache would hold defines the tensors; it also makes a
second identical query reproduce the first bit for bit).  `round_cache=False` removes that single rounding and is
what pins this file to the plain dense decoder.  Block structure as in oracle/reuse_prefill.py (pre-norm RMSNorm,
half-split RoPE, GQA by contiguous groups, SwiGLU, no biases, no final norm); its leaf functions (rmsnorm, rope,
silu, round_to_bf16) are reused, the attention here is written out with an explicit lower-triangular mask.

Pins (tests/test_oracle_paper_mode.py): without rounding and with an empty cache it equals dense_prefill on every
row; with rounding, a prompt served from any matched prefix (with or without tail drop) equals the same prompt
served from an empty cache; cached tensors are bf16-representable and are the in-context slices; L_pre and the
matched chain by hand; the new rows agree with reuse_prefill's prefix mode up to the placement of the rounding.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from oracle.reuse_prefill import Model, rmsnorm, rope, round_to_bf16, silu


@dataclass
class PaperPrompt:
    chunk_ids: Sequence[int]
    chunk_len: Sequence[int]
    chunk_hidden: Sequence[np.ndarray]        # float64 [len, d] for EVERY chunk: the whole prompt is embedded
    query_hidden: np.ndarray                  # float64 [n_query, d]
    tail_drop: int = 0                        # tokens of the final matched node to recompute


class PaperStore:
    """path of chunk ids (tuple) -> (Q, K, V): float64 [n_layers, n_tokens, heads, hd] holding the cached values;
    Q and K after position encoding at the positions the node has on its path."""

    def __init__(self):
        self.qkv: Dict[Tuple[int, ...], Tuple[np.ndarray, np.ndarray, np.ndarray]] = {}

    def has(self, path) -> bool:
        return tuple(path) in self.qkv


@dataclass
class PaperResult:
    n_matched: int                 # chunks of the matched chain
    l_pre: int                     # rows served from the cache (Appendix B.1)
    l_total: int
    out_hidden: np.ndarray         # float64 [l_total, d]


def match_chain(store: PaperStore, prompt: PaperPrompt) -> Tuple[int, int]:
    """(number of matched chunks, L_pre): walk the tree from the first chunk until the first mismatch; the final
    matched node gives up its last tail_drop tokens."""
    n = 0
    while n < len(prompt.chunk_ids) and store.has(prompt.chunk_ids[: n + 1]):
        stored = store.qkv[tuple(prompt.chunk_ids[: n + 1])][0].shape[1]
        if stored != prompt.chunk_len[n]:
            raise ValueError(f"node {tuple(prompt.chunk_ids[: n + 1])}: stored {stored} tokens, prompt says {prompt.chunk_len[n]}")
        n += 1
    l_pre = int(sum(prompt.chunk_len[:n]))
    drop = int(prompt.tail_drop or 0)
    if drop < 0 or (n > 0 and drop > prompt.chunk_len[n - 1]):
        raise ValueError("tail_drop must lie between 0 and the length of the final matched chunk")
    if n > 0:
        l_pre -= drop
    return n, l_pre


def paper_prefill(model: Model, store: PaperStore, prompts: Sequence[PaperPrompt], commit: bool = True,
                  round_cache: bool = True) -> List[PaperResult]:
    """Prefill with the paper's QKV cache: all L_total rows leave every block, the first L_pre skip the projections."""
    hq, hkv, hd = model.n_q_heads, model.n_kv_heads, model.head_dim
    group = hq // hkv
    plans = [match_chain(store, p) for p in prompts]          # against the store as it is when the call starts
    results: List[PaperResult] = []
    pending = []
    for prompt, (n_match, l_pre) in zip(prompts, plans):
        x = np.concatenate([np.asarray(h, dtype=np.float64) for h in prompt.chunk_hidden] +
                           [np.asarray(prompt.query_hidden, dtype=np.float64)], axis=0)      # embedding output
        T = x.shape[0]
        # the loaded chain, concatenated in order, cut to L_pre rows
        if n_match:
            lq = np.concatenate([store.qkv[tuple(prompt.chunk_ids[: i + 1])][0] for i in range(n_match)], axis=1)[:, :l_pre]
            lk = np.concatenate([store.qkv[tuple(prompt.chunk_ids[: i + 1])][1] for i in range(n_match)], axis=1)[:, :l_pre]
            lv = np.concatenate([store.qkv[tuple(prompt.chunk_ids[: i + 1])][2] for i in range(n_match)], axis=1)[:, :l_pre]
        pos_new = np.arange(l_pre, T)                          # position counter offset by L_pre
        causal = np.tril(np.ones((T, T), dtype=bool))
        q_layers, k_layers, v_layers = [], [], []
        for l in range(model.n_layers):
            xc = x[l_pre:]                                     # crop the first L_pre rows of the block's input
            xn = rmsnorm(xc, model.w(l, "attn_norm"), model.rms_eps)
            q = rope((xn @ model.w(l, "wq").T).reshape(T - l_pre, hq, hd), pos_new, model.rope_theta)
            k = rope((xn @ model.w(l, "wk").T).reshape(T - l_pre, hkv, hd), pos_new, model.rope_theta)
            v = (xn @ model.w(l, "wv").T).reshape(T - l_pre, hkv, hd)
            if round_cache:
                q, k, v = round_to_bf16(q), round_to_bf16(k), round_to_bf16(v)
            if n_match:                                        # loaded tensors in front: length back to L_total
                q = np.concatenate([lq[l], q], axis=0)
                k = np.concatenate([lk[l], k], axis=0)
                v = np.concatenate([lv[l], v], axis=0)
            q_layers.append(q)
            k_layers.append(k)
            v_layers.append(v)
            att = np.empty((T, hq, hd), dtype=np.float64)      # "the subsequent operations proceed normally"
            for h in range(hq):
                s = q[:, h, :] @ k[:, h // group, :].T / np.sqrt(float(hd))
                s = np.where(causal, s, -np.inf)
                e = np.exp(s - s.max(axis=1, keepdims=True))
                att[:, h, :] = (e / e.sum(axis=1, keepdims=True)) @ v[:, h // group, :]
            x = x + att.reshape(T, hq * hd) @ model.w(l, "wo").T
            yn = rmsnorm(x, model.w(l, "ffn_norm"), model.rms_eps)
            x = x + (silu(yn @ model.w(l, "w_gate").T) * (yn @ model.w(l, "w_up").T)) @ model.w(l, "w_down").T
        # slice the collected tensors per chunk on the sequence axis; nodes of the matched chain already exist
        start = int(sum(prompt.chunk_len[:n_match]))
        for i in range(n_match, len(prompt.chunk_ids)):
            n = prompt.chunk_len[i]
            pending.append((tuple(prompt.chunk_ids[: i + 1]),
                            np.stack([t[start:start + n] for t in q_layers]),
                            np.stack([t[start:start + n] for t in k_layers]),
                            np.stack([t[start:start + n] for t in v_layers])))
            start += n
        results.append(PaperResult(n_match, l_pre, T, x))
    if commit:
        for path, qs, ks, vs in pending:
            if path not in store.qkv:
                store.qkv[path] = (qs, ks, vs)
    return results
