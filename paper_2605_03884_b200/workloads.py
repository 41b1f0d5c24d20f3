"""Seeded synthetic inputs for the CacheCard create / inject path.

This module holds *only* input generation: FP16 KV caches with the shapes and value
distributions of the benchmark configurations, per-token bit-width vectors drawn at random, and
importance scores.  It contains none of the method's arithmetic (no quantisation, packing,
offsets, sizes or rank rule), so both the
CUDA path and the CPU oracle can be fed from it without sharing any code of the method.

The synthetic caches stand in for real Llama-3.1-8B-Instruct KV caches (Section 5.1 of the
paper): values are drawn N(0,1) in fp32 and rounded to FP16; keys additionally carry four
fixed outlier channels per (layer, head), scaled by 10, which models the channel-wise key
outliers that per-channel key quantisers are built around (Section 2 related work).
The bit-width vectors stand in for the output of the paper's bit-allocation controller
(Section 4.1.2), which needs trained weights and attention statistics that do not exist here.

Seeds (fixed so every run sees the same bytes):
  values            seed          (0 for config 1, 1000 + config number otherwise;
                                   config 5 starts from config 3's cache, seed 1003)
  outlier channels  seed + 1      rng.choice(d, 4, replace=False) per (layer, head)
  i.i.d. bits       seed + 2
  importance score  seed + 3      LogNormal(0, 1) per token (config 4)
  chain hop k bits  seed + 10 + k (config 5; seed 1005)
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Callable, Iterator, Optional, Tuple

import numpy as np

BIT_CHOICES = np.array([2, 4, 8, 16], dtype=np.uint8)


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shape + distributions + bit-width recipe)."""

    name: str
    number: int
    n_layers: int
    n_kv_heads: int
    head_dim: int
    n_tokens: int
    value_seed: int
    k_outliers: int            # outlier channels per (layer, head) in K, scaled x10
    bits_recipe: str           # "uniform4" | "iid" | "quantile" | "chain"
    iid_probs: Tuple[float, float, float, float] = (0.0, 1.0, 0.0, 0.0)
    hops: int = 1

    @property
    def n_streams(self) -> int:
        return 2 * self.n_layers * self.n_kv_heads

    @property
    def kv_bytes(self) -> int:
        return self.n_streams * self.n_tokens * self.head_dim * 2

    def scaled(self, **kw) -> "Workload":
        """Same recipe at another shape (used for CPU-sized test cases)."""
        return replace(self, **kw)


WORKLOADS = {
    1: Workload("tiny_uniform4", 1, 1, 2, 64, 128, 0, 0, "uniform4"),
    2: Workload("llama8b_1k_mixed", 2, 32, 8, 128, 1024, 1002, 4, "iid",
                iid_probs=(0.40, 0.40, 0.15, 0.05)),
    3: Workload("llama8b_8k_uniform4", 3, 32, 8, 128, 8192, 1003, 4, "uniform4"),
    4: Workload("llama8b_8k_adaptive", 4, 32, 8, 128, 8192, 1004, 4, "quantile"),
    5: Workload("llama8b_8k_chain4", 5, 32, 8, 128, 8192, 1003, 4, "chain",
                iid_probs=(0.30, 0.40, 0.20, 0.10), hops=4),
}


def outlier_channels(w: Workload) -> np.ndarray:
    """[n_layers, n_kv_heads, k_outliers] channel indices, fixed across tokens."""
    rng = np.random.default_rng(w.value_seed + 1)
    out = np.zeros((w.n_layers, w.n_kv_heads, max(w.k_outliers, 0)), dtype=np.int64)
    for l in range(w.n_layers):
        for h in range(w.n_kv_heads):
            if w.k_outliers:
                out[l, h] = rng.choice(w.head_dim, w.k_outliers, replace=False)
    return out


def kv_layers(w: Workload, layers: Optional[range] = None
              ) -> Iterator[Tuple[int, np.ndarray, np.ndarray]]:
    """Yield (layer, K, V) with K, V FP16 arrays of shape [n_kv_heads, n_tokens, head_dim].

    Layers are always drawn in order from one generator so that layer l holds the same bytes
    whether or not a caller consumes the layers before it; `layers` only selects what is
    yielded.
    """
    rng = np.random.default_rng(w.value_seed)
    ch = outlier_channels(w)
    shape = (w.n_kv_heads, w.n_tokens, w.head_dim)
    want = set(range(w.n_layers) if layers is None else layers)
    last = max(want) if want else -1
    for l in range(w.n_layers):
        if l > last:
            break
        k = rng.standard_normal(shape, dtype=np.float32)
        v = rng.standard_normal(shape, dtype=np.float32)
        if l not in want:
            continue
        for h in range(w.n_kv_heads):
            if w.k_outliers:
                k[h][:, ch[l, h]] *= np.float32(10.0)
        yield l, k.astype(np.float16), v.astype(np.float16)


def iid_bits(n_tokens: int, probs, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed)
    idx = rng.choice(4, size=n_tokens, p=np.asarray(probs, dtype=np.float64))
    return BIT_CHOICES[idx]


def importance_scores(n_tokens: int, seed: int) -> np.ndarray:
    """Synthetic per-token importance (config 4): LogNormal(0, 1), float32."""
    rng = np.random.default_rng(seed)
    return rng.lognormal(0.0, 1.0, size=n_tokens).astype(np.float32)


def quantile_counts(n_tokens: int) -> Tuple[int, int, int]:
    """How many tokens the adaptive recipe keeps in FP16, at 8 bits and at 4 bits (the rest get
    2 bits): top 5 %, next 15 %, next 40 %, with the cut ranks rounded half-up from 0.05 T, 0.20 T
    and 0.60 T (410 / 1228 / 3277 of 8192)."""
    c16 = int(np.floor(0.05 * n_tokens + 0.5))
    c8 = int(np.floor(0.20 * n_tokens + 0.5))
    c4 = int(np.floor(0.60 * n_tokens + 0.5))
    return c16, c8 - c16, c4 - c8


RankRule = Callable[[np.ndarray, int, int, int], np.ndarray]


def bits_for(w: Workload, hop: int = 0, segment: int = 0, rank_rule: Optional[RankRule] = None) -> np.ndarray:
    """Per-token bit-width vector (uint8, values in {2,4,8,16}; 16 means raw FP16).  `segment`
    varies the draw for the per-(layer, head) mode; segment 0 is the whole-model vector.

    The adaptive recipe ("quantile") only draws the importance scores here; turning scores into
    bit-widths by rank is a step of the method, so the caller supplies it as
    `rank_rule(scores, n_fp16, n_8bit, n_4bit) -> bits`: the library's entry point, the oracle's
    function, or a test's own statement of the rule."""
    t = w.n_tokens
    shift = 7919 * segment
    if w.bits_recipe == "uniform4":
        return np.full(t, 4, dtype=np.uint8)
    if w.bits_recipe == "iid":
        return iid_bits(t, w.iid_probs, w.value_seed + 2 + shift)
    if w.bits_recipe == "quantile":
        if rank_rule is None:
            raise ValueError("the adaptive recipe needs a rank_rule (scores, n_fp16, n_8bit, n_4bit) -> bits")
        bits = np.asarray(rank_rule(importance_scores(t, w.value_seed + 3 + shift), *quantile_counts(t)), dtype=np.uint8)
        assert bits.shape == (t,)
        return bits
    if w.bits_recipe == "chain":
        return iid_bits(t, w.iid_probs, 1000 + w.number + 10 + hop + shift)
    raise ValueError(w.bits_recipe)


def bits_per_head(w: Workload, hop: int = 0, rank_rule: Optional[RankRule] = None) -> np.ndarray:
    """bits[n_layers * n_kv_heads][n_tokens], flattened: every (layer, head) segment draws the
    workload's recipe on its own (as a controller that scores tokens per head would)."""
    return np.concatenate([bits_for(w, hop, seg, rank_rule) for seg in range(w.n_layers * w.n_kv_heads)])


def random_fp16(shape, seed: int, scale: float = 1.0) -> np.ndarray:
    """Plain N(0, scale^2) FP16 block for small ad-hoc test cases."""
    rng = np.random.default_rng(seed)
    return (rng.standard_normal(shape, dtype=np.float32) * np.float32(scale)).astype(np.float16)
