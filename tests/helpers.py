"""Glue between the seeded input generators and the CPU oracle (tests only)."""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np

from oracle import reuse_prefill as orc
from paper_2601_11553_b200 import workloads as wl


def oracle_model(shape: wl.ModelShape, weights: List[dict]) -> orc.Model:
    return orc.Model(n_layers=shape.n_layers, d_model=shape.d_model, n_q_heads=shape.n_q_heads,
                     n_kv_heads=shape.n_kv_heads, head_dim=shape.head_dim, d_ffn=shape.d_ffn,
                     rope_theta=shape.rope_theta, rms_eps=shape.rms_eps, layers=weights)


def oracle_prompt(p: wl.Prompt, drop_hidden_of: Sequence[int] = ()) -> orc.Prompt:
    hid: List[Optional[np.ndarray]] = []
    for i, h in enumerate(p.chunk_hidden):
        hid.append(None if (i in drop_hidden_of or h is None) else orc.bf16_bits_to_f64(h))
    if not p.chunk_hidden:
        hid = [None] * len(p.chunk_ids)
    return orc.Prompt(chunk_ids=list(p.chunk_ids), chunk_len=list(p.chunk_len), chunk_hidden=hid,
                      query_hidden=orc.bf16_bits_to_f64(p.query_hidden))


def concat_hidden(p: wl.Prompt) -> np.ndarray:
    parts = [orc.bf16_bits_to_f64(h) for h in p.chunk_hidden] + [orc.bf16_bits_to_f64(p.query_hidden)]
    return np.concatenate(parts, axis=0)


def populate_alone(model: orc.Model, store: orc.Store, seed: int, chunk_id: int, n_tokens: int) -> None:
    """Store a chunk by prefilling it alone (no hits, no query tokens)."""
    h = orc.bf16_bits_to_f64(wl.chunk_hidden_for(seed, chunk_id, n_tokens, model.d_model))
    pr = orc.Prompt([chunk_id], [n_tokens], [h], np.zeros((0, model.d_model)))
    orc.reuse_prefill(model, store, [pr])
