"""CPU definition of the QA-bank lookup.  TEST INFRASTRUCTURE ONLY (see oracle/reuse_prefill.py).

Paper Section 3.4.1 ("Similar Query Reuse"): the query embedding is compared by cosine similarity with all
stored query embeddings; if the highest similarity exceeds tau_query the stored answer is returned.
Float64 throughout; among equal maxima the lowest index is taken.
"""
from __future__ import annotations

import numpy as np


def cosine_scores(bank: np.ndarray, queries: np.ndarray) -> np.ndarray:
    """scores[q, i] = <queries[q], bank[i]> / (|queries[q]| |bank[i]|)."""
    b = np.asarray(bank, dtype=np.float64)
    q = np.asarray(queries, dtype=np.float64)
    bn = np.sqrt(np.sum(b * b, axis=1))
    qn = np.sqrt(np.sum(q * q, axis=1))
    return (q @ b.T) / (qn[:, None] * bn[None, :])


def top1(bank: np.ndarray, queries: np.ndarray, tau_query: float):
    s = cosine_scores(bank, queries)
    idx = np.argmax(s, axis=1)                 # first occurrence of the maximum = lowest index
    best = s[np.arange(s.shape[0]), idx]
    return idx.astype(np.int32), best, (best > tau_query).astype(np.uint8), s
