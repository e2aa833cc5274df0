"""Seeded synthetic inputs for reuse-prefill: model shapes, weights, prompts, hit masks.

This module only *draws inputs*.  It holds none of the method's arithmetic (no
norm, projection, rotation, attention or cache assembly), so both the CUDA
binding's tests and the CPU oracle's tests may import it without sharing any
computation.  Everything is a pure function of an integer seed.

Values are produced as bf16 bit patterns (``uint16``): the library's weight and
hidden-state inputs are bf16, and a checker can widen the very same bits to any
wider float type without a second rounding.

The prompts take the shape of the mobile-RAG prompts the paper describes
(Section 3.2 "Cache Architecture": system prompt + retrieved knowledge chunks +
user query; Appendix A.4: chunks of 100 words; Section 5.7: a 349-token input)
scaled up as the five workload descriptions direct.  They stand in for the
paper's datasets, none of whose items is reproduced here.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

PAGE_TOKENS = 16


# --------------------------------------------------------------------------- #
# bf16 bit helpers (format conversion only)
# --------------------------------------------------------------------------- #
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 values to bf16 (nearest, ties to even); return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- #
# model shape and weights
# --------------------------------------------------------------------------- #
@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    rope_theta: float = 1.0e6
    rms_eps: float = 1.0e-6

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def params_per_layer(self) -> int:
        d, f = self.d_model, self.d_ffn
        return d * (self.q_dim + 2 * self.kv_dim) + self.q_dim * d + 3 * d * f


SHAPE_A = dict(d_model=1024, n_q_heads=16, n_kv_heads=8, head_dim=128, d_ffn=3072)
SHAPE_B = dict(d_model=2048, n_q_heads=16, n_kv_heads=8, head_dim=128, d_ffn=5632)

WEIGHT_NAMES = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")


def weight_shapes(shape: ModelShape) -> Dict[str, tuple]:
    """[out_features, in_features] of every projection matrix of one layer."""
    d, f = shape.d_model, shape.d_ffn
    return {
        "wq": (shape.q_dim, d), "wk": (shape.kv_dim, d), "wv": (shape.kv_dim, d),
        "wo": (d, shape.q_dim), "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f),
    }


def make_layer_weights(shape: ModelShape, seed: int, layer: int, std: float = 0.02,
                       random_gains: bool = False) -> Dict[str, np.ndarray]:
    """bf16 bit patterns of one layer's weights: projections ~ N(0, std); norm gains = 1 as the workload
    descriptions say, or, with random_gains, 1 + 0.3 N(0, 1) per element and norm (for checks that must notice a
    gain that is dropped, swapped between the two norms, or read at the wrong index)."""
    out: Dict[str, np.ndarray] = {}
    for i, (name, shp) in enumerate(weight_shapes(shape).items()):
        rng = np.random.default_rng([seed, 7001, layer, i])
        w = rng.standard_normal(shp, dtype=np.float32) * np.float32(std)
        out[name] = f32_to_bf16_bits(w)
    for j, name in enumerate(("attn_norm", "ffn_norm")):
        g = np.ones(shape.d_model, dtype=np.float32)
        if random_gains:
            g = g + np.float32(0.3) * np.random.default_rng([seed, 7006, layer, j]).standard_normal(
                shape.d_model, dtype=np.float32)
        out[name] = f32_to_bf16_bits(g)
    return out


def make_weights(shape: ModelShape, seed: int, std: float = 0.02, random_gains: bool = False) -> List[Dict[str, np.ndarray]]:
    return [make_layer_weights(shape, seed, l, std, random_gains) for l in range(shape.n_layers)]


def make_hidden(seed: int, tag: Sequence[int], n_tokens: int, d_model: int) -> np.ndarray:
    """bf16 bit patterns [n_tokens, d_model] of N(0, 1) hidden states for one chunk / query."""
    rng = np.random.default_rng([seed, 7002, *[int(t) for t in tag]])
    return f32_to_bf16_bits(rng.standard_normal((n_tokens, d_model), dtype=np.float32))


# --------------------------------------------------------------------------- #
# prompts
# --------------------------------------------------------------------------- #
@dataclass
class Prompt:
    """An ordered list of chunk IDs plus new query tokens (paper Section 3, system overview)."""
    chunk_ids: List[int]
    chunk_len: List[int]
    n_query: int
    # bf16 bits; chunk_hidden[i] is [chunk_len[i], d]; hidden depends on the chunk id only.
    chunk_hidden: List[np.ndarray] = field(default_factory=list)
    query_hidden: Optional[np.ndarray] = None

    @property
    def n_total(self) -> int:
        return int(sum(self.chunk_len) + self.n_query)


@dataclass
class Workload:
    name: str
    shape: ModelShape
    seed: int
    prompts: List[Prompt]
    # chunk ids that are in the cache before the timed / checked call
    cached_ids: List[int]
    description: str = ""
    # how the cached K/V of `cached_ids` is produced:
    #   "prefill_alone"  : prefill each cached chunk alone (no hits, no query) and keep what it stores
    #   "same_inputs_l1" : single layer; K/V from the same chunk hidden states (any method agrees)
    #   "integer_pool"   : counter-based integer generator (pool_kv_values)
    cache_source: str = "prefill_alone"
    # True: chunks are matched as a path of the cache tree (the paper's rule); cached_ids then is a prefix of the list
    # and the cached content comes from a prefill of exactly that prefix ("prefill_prefix")
    match_prefix: bool = False
    # True: the paper-faithful mode of the library (cached Q as well, every row of the prompt continues)
    paper_mode: bool = False

    @property
    def total_tokens(self) -> int:
        return sum(p.n_total for p in self.prompts)

    def new_rows(self) -> int:
        cached = set(self.cached_ids)
        n = 0
        for p in self.prompts:
            n += p.n_query + sum(l for c, l in zip(p.chunk_ids, p.chunk_len) if c not in cached)
        return n


def chunk_hidden_for(seed: int, chunk_id: int, n_tokens: int, d_model: int) -> np.ndarray:
    return make_hidden(seed, (1, chunk_id), n_tokens, d_model)


def _single_prompt(shape: ModelShape, seed: int, n_chunks: int, chunk_tokens, n_query: int,
                   id_base: int = 0, with_hidden: bool = True) -> Prompt:
    lens = [int(chunk_tokens)] * n_chunks if np.isscalar(chunk_tokens) else [int(c) for c in chunk_tokens]
    ids = [id_base + i for i in range(n_chunks)]
    p = Prompt(chunk_ids=ids, chunk_len=lens, n_query=int(n_query))
    if with_hidden:
        p.chunk_hidden = [chunk_hidden_for(seed, c, l, shape.d_model) for c, l in zip(ids, lens)]
        p.query_hidden = make_hidden(seed, (2, 0), n_query, shape.d_model)
    return p


def exact_hit_set(n_chunks: int, n_hits: int, seed: int) -> List[int]:
    """Indices of exactly n_hits chunks, placed by a seeded permutation."""
    perm = np.random.default_rng([seed, 7003]).permutation(n_chunks)
    return sorted(int(i) for i in perm[:n_hits])


def bernoulli_hit_set(n_chunks: int, p: float, seed: int) -> List[int]:
    u = np.random.default_rng([seed, 7004]).random(n_chunks)
    return [int(i) for i in range(n_chunks) if u[i] < p]


def zipf_ids_no_repeat(rng: np.random.Generator, n: int, pool: int, alpha: float) -> List[int]:
    """n distinct ids from {0..pool-1}, drawn with P(id = k) ∝ (k+1)^-alpha, redrawing repeats."""
    w = 1.0 / np.power(np.arange(1, pool + 1, dtype=np.float64), alpha)
    cdf = np.cumsum(w / w.sum())
    seen: List[int] = []
    s = set()
    while len(seen) < n:
        k = int(np.searchsorted(cdf, rng.random(), side="right"))
        k = min(k, pool - 1)
        if k not in s:
            s.add(k)
            seen.append(k)
    return seen


def config0(with_hidden: bool = True) -> Workload:
    """One layer of shape A; 4 x 128 + 32 = 544 tokens; all four chunks hit."""
    shape = ModelShape(n_layers=1, **SHAPE_A)
    p = _single_prompt(shape, 0, 4, 128, 32, with_hidden=with_hidden)
    return Workload("cfg0", shape, 0, [p], cached_ids=list(p.chunk_ids), cache_source="same_inputs_l1",
                    description="1 layer, 4x128+32=544 tokens, all chunks hit")


def config1(with_hidden: bool = True) -> Workload:
    """28 layers of shape A; 8 x 256 + 64 = 2112 tokens; Bernoulli(0.5) hit mask."""
    shape = ModelShape(n_layers=28, **SHAPE_A)
    p = _single_prompt(shape, 1, 8, 256, 64, with_hidden=with_hidden)
    hits = bernoulli_hit_set(8, 0.5, 1)
    return Workload("cfg1", shape, 1, [p], cached_ids=[p.chunk_ids[i] for i in hits],
                    description="28 layers, 8x256+64=2112 tokens, Bernoulli(0.5) per-chunk hits")


def config2(with_hidden: bool = True) -> Workload:
    """16 layers of shape B; 16 x 512 + 128 = 8320 tokens; exactly 12 of 16 chunks hit."""
    shape = ModelShape(n_layers=16, **SHAPE_B)
    p = _single_prompt(shape, 2, 16, 512, 128, with_hidden=with_hidden)
    hits = exact_hit_set(16, 12, 2)
    return Workload("cfg2", shape, 2, [p], cached_ids=[p.chunk_ids[i] for i in hits],
                    description="16 layers d=2048, 16x512+128=8320 tokens, 12/16 chunks hit")


def config3(with_hidden: bool = True, n_prompts: int = 64, pool: int = 4096, n_layers: int = 28) -> Workload:
    """Batched serving on the config-1 model: ragged prompts over a Zipf(1.1) pool of cached chunks."""
    shape = ModelShape(n_layers=n_layers, **SHAPE_A)
    rng = np.random.default_rng([3, 7005])
    prompts: List[Prompt] = []
    used = set()
    for b in range(n_prompts):
        nc = int(rng.integers(2, 17))
        nq = int(rng.integers(32, 129))
        ids = zipf_ids_no_repeat(rng, nc, pool, 1.1)
        p = Prompt(chunk_ids=ids, chunk_len=[256] * nc, n_query=nq)
        if with_hidden:
            p.query_hidden = make_hidden(3, (2, b), nq, shape.d_model)
            p.chunk_hidden = []          # every chunk is expected to hit; no hidden needed
        prompts.append(p)
        used.update(ids)
    return Workload("cfg3", shape, 3, prompts, cached_ids=sorted(used), cache_source="integer_pool",
                    description=f"{n_prompts} prompts, 2-16 chunks x 256 + 32-128 query, Zipf(1.1) ids over {pool}")


def config4(hit_rate: float, with_hidden: bool = True) -> Workload:
    """Long context on the config-1 model: 64 x 512 + 256 = 33024 tokens; exact hit count."""
    shape = ModelShape(n_layers=28, **SHAPE_A)
    p = _single_prompt(shape, 4, 64, 512, 256, with_hidden=with_hidden)
    n_hits = int(round(hit_rate * 64))
    hits = exact_hit_set(64, n_hits, 4)
    return Workload(f"cfg4_{int(round(hit_rate * 100))}", shape, 4, [p],
                    cached_ids=[p.chunk_ids[i] for i in hits],
                    description=f"28 layers, 64x512+256=33024 tokens, {n_hits}/64 chunks hit")


def prefix_config1(paper_mode: bool, with_hidden: bool = True) -> Workload:
    """The 28-layer workload's prompt (8 x 256 + 64 tokens) with the first four chunks cached as a chain of the cache
    tree: the case the paper itself reuses.  Run in the library's default reading (only the 1088 new rows continue)
    or in the paper-faithful mode (all 2112 rows continue, the cached ones skip the projections)."""
    shape = ModelShape(n_layers=28, **SHAPE_A)
    p = _single_prompt(shape, 1, 8, 256, 64, with_hidden=with_hidden)
    return Workload("paper_cfg1" if paper_mode else "prefix_cfg1", shape, 1, [p], cached_ids=list(p.chunk_ids[:4]),
                    cache_source="prefill_prefix", match_prefix=True, paper_mode=paper_mode,
                    description="28 layers, 8x256+64=2112 tokens, first 4 chunks cached as a prefix chain"
                                + (", paper-faithful mode (all rows continue)" if paper_mode else ", new rows only"))


def by_name(name: str, with_hidden: bool = True) -> Workload:
    if name == "prefix_cfg1":
        return prefix_config1(False, with_hidden)
    if name == "paper_cfg1":
        return prefix_config1(True, with_hidden)
    if name == "cfg0":
        return config0(with_hidden)
    if name == "cfg1":
        return config1(with_hidden)
    if name == "cfg2":
        return config2(with_hidden)
    if name == "cfg3":
        return config3(with_hidden)
    if name.startswith("cfg4_"):
        return config4(int(name.split("_")[1]) / 100.0, with_hidden)
    raise KeyError(name)


def small_workload(seed: int, n_layers: int, chunk_lens: Sequence[int], n_query: int, hit_idx: Sequence[int],
                   d_model: int = 256, n_q_heads: int = 4, n_kv_heads: int = 2, head_dim: int = 128,
                   d_ffn: int = 512, id_base: int = 100) -> Workload:
    """A reduced model for element-by-element checks; ragged chunk lengths allowed."""
    shape = ModelShape(n_layers=n_layers, d_model=d_model, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads,
                       head_dim=head_dim, d_ffn=d_ffn)
    p = _single_prompt(shape, seed, len(chunk_lens), list(chunk_lens), n_query, id_base=id_base)
    return Workload(f"small{seed}", shape, seed, [p], cached_ids=[p.chunk_ids[i] for i in hit_idx],
                    description="reduced model")


# --------------------------------------------------------------------------- #
# counter-based integer pool values (config 3)
# --------------------------------------------------------------------------- #
_M64 = (1 << 64) - 1


def splitmix64(x: np.ndarray) -> np.ndarray:
    """The SplitMix64 output function (Steele, Lea, Flood 2014) applied to uint64 counters."""
    with np.errstate(over="ignore"):
        z = (x + np.uint64(0x9E3779B97F4A7C15)).astype(np.uint64)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def pool_kv_values(seed: int, chunk_id: int, which: int, layer: int, n_tokens: int, kv_dim: int) -> np.ndarray:
    """Synthetic pre-RoPE K (which=0) or V (which=1) of a pooled chunk, bf16 bits [n_tokens, kv_dim].

    Element e of (chunk, which, layer) takes counter
        c = ((((seed * 2^20 + chunk_id) * 2 + which) * 64 + layer) << 24) + e
    and value (b0 + b1 + b2 + b3 - 126) / 64 with b_i the four lowest 6-bit fields of
    splitmix64(c): multiples of 1/64 in [-1.97, 1.97], exactly representable in bf16.
    """
    base = ((((seed << 20) + chunk_id) * 2 + which) * 64 + layer) << 24
    e = np.arange(n_tokens * kv_dim, dtype=np.uint64) + np.uint64(base & _M64)
    h = splitmix64(e)
    s = np.zeros(e.shape, dtype=np.int64)
    for i in range(4):
        s += ((h >> np.uint64(6 * i)) & np.uint64(63)).astype(np.int64)
    v = (s - 126).astype(np.float32) / np.float32(64.0)
    return f32_to_bf16_bits(v).reshape(n_tokens, kv_dim)
