"""CPU oracle for the decode step that follows reuse-prefill.  TEST INFRASTRUCTURE ONLY.

Imported by the tests (and the smoke check); the product never routes through it and it shares no
code with the CUDA path.

What it computes: after the prompt has been prefilled (paper Section 2.1: inference is a prefill stage
over the whole prompt followed by a decode stage that produces one token at a time, each step attending
to the keys and values of everything before it), one more token is appended at position T.  Its hidden
state goes through every block: RMSNorm, Q/K/V projection, K and V rounded to the cache format, K and Q
rotated to position T, attention of the single row over slots 0..T (the assembled context of the
prefill plus the token itself), output projection, SwiGLU FFN.  The token's rotated K and its V join the
context, so the next step sees T + 1 slots.

The definition has a plain equivalent that pins it (tests/test_oracle_decode.py): prefilling the prompt
with the token appended to the query gives, in its last row, the same output, and an ordinary dense
causal decoder over the whole sequence does too when nothing was cached.

Arithmetic is float64 (numpy); the one rounding is K/V -> bf16, as in the prefill oracle.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

import numpy as np

from oracle.reuse_prefill import Model, PromptResult, attention_rows, rmsnorm, rope, round_to_bf16, silu


@dataclass
class DecodeState:
    """Per layer: rotated K and V of every slot so far, float64 [T, Hkv, hd] (bf16 values before rotation)."""
    k_ctx: List[np.ndarray]
    v_ctx: List[np.ndarray]

    @property
    def n_tokens(self) -> int:
        return int(self.k_ctx[0].shape[0])


def begin_decode(result: PromptResult) -> DecodeState:
    """State after a prefill that was asked to keep its assembled context (keep_ctx=True)."""
    if result.k_ctx is None or result.v_ctx is None:
        raise ValueError("prefill result holds no assembled context: call reuse_prefill(..., keep_ctx=True)")
    return DecodeState([np.array(k) for k in result.k_ctx], [np.array(v) for v in result.v_ctx])


def decode_step(model: Model, state: DecodeState, hidden: np.ndarray) -> np.ndarray:
    """One token: hidden [d] (float64) at position T = state.n_tokens; returns its final residual [d].

    The state grows by the token's rotated K and its V in every layer.
    """
    hq, hkv, hd = model.n_q_heads, model.n_kv_heads, model.head_dim
    T = state.n_tokens
    pos = np.array([T])
    x = np.array(hidden, dtype=np.float64).reshape(1, model.d_model)
    for l in range(model.n_layers):
        xn = rmsnorm(x, model.w(l, "attn_norm"), model.rms_eps)
        q = (xn @ model.w(l, "wq").T).reshape(1, hq, hd)
        k = round_to_bf16((xn @ model.w(l, "wk").T).reshape(1, hkv, hd))       # what a cache would hold
        v = round_to_bf16((xn @ model.w(l, "wv").T).reshape(1, hkv, hd))
        state.k_ctx[l] = np.concatenate([state.k_ctx[l], rope(k, pos, model.rope_theta)], axis=0)
        state.v_ctx[l] = np.concatenate([state.v_ctx[l], v], axis=0)
        att = attention_rows(rope(q, pos, model.rope_theta), pos, state.k_ctx[l], state.v_ctx[l])
        x = x + att @ model.w(l, "wo").T
        yn = rmsnorm(x, model.w(l, "ffn_norm"), model.rms_eps)
        x = x + (silu(yn @ model.w(l, "w_gate").T) * (yn @ model.w(l, "w_up").T)) @ model.w(l, "w_down").T
    return x[0]
