"""Seeded partitions, class masks and logits shaped like the paper's workloads.

Vocabulary sizes and class counts follow the paper's Table 1 (V = 128256 and
151936; K from about 256 to a few thousand); the tokenizers, grammars and
datasets themselves are not available, so class sizes are drawn from a
Zipf-like law and members are scattered over the vocabulary by a seeded
shuffle. Everything here is an input recipe: nothing computes an expansion,
a masking or a reduction.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

from . import rng

# stream purposes
_P_RANKS, _P_SHUFFLE, _P_MASK, _P_LOGITS, _P_SPIKES, _P_DENSITY, _P_NCLS, _P_UNIFORM = 1, 2, 3, 4, 5, 6, 7, 8


@dataclass
class Partition:
    """token -> class vector ``c`` (int32 [V]) and class -> representative vector ``r`` (int32 [K])."""

    V: int
    K: int
    c: np.ndarray
    r: np.ndarray
    sizes: np.ndarray  # int64 [K], number of tokens per class


def _largest_remainder(total: int, weights: np.ndarray) -> np.ndarray:
    """Split ``total`` units proportionally to ``weights`` (largest-remainder rounding)."""
    if total <= 0:
        return np.zeros(len(weights), dtype=np.int64)
    q = weights / weights.sum() * total
    base = np.floor(q).astype(np.int64)
    left = int(total - base.sum())
    if left > 0:
        order = np.argsort(-(q - base), kind="stable")
        base[order[:left]] += 1
    return base


def _partition_from_sizes(V: int, sizes: np.ndarray, shuffle_key) -> Partition:
    K = len(sizes)
    assert int(sizes.sum()) == V and int(sizes.min()) >= 1
    labels = np.repeat(np.arange(K, dtype=np.int32), sizes)
    perm = rng.permutation(shuffle_key, V)
    c = np.empty(V, dtype=np.int32)
    c[perm] = labels  # token perm[j] gets label j: members scattered over the vocabulary
    r = np.full(K, V, dtype=np.int64)
    np.minimum.at(r, c, np.arange(V, dtype=np.int64))  # representative = lowest token id in the class
    return Partition(V=V, K=K, c=c, r=r.astype(np.int32), sizes=sizes.astype(np.int64))


def zipf_partition(V: int, K: int, s: float = 1.1, seed: int = 0, config: int = 0) -> Partition:
    """Every class non-empty; the V-K remaining tokens are split ~ rank^-s over size ranks.

    Size ranks are assigned to class ids by a seeded permutation, so class 0 is
    not always the largest class.
    """
    assert 1 <= K <= V
    w = np.arange(1, K + 1, dtype=np.float64) ** (-s)
    by_rank = 1 + _largest_remainder(V - K, w)
    ranks = rng.permutation(rng.stream_key(rng.SEED_BASE, config, _P_RANKS, seed), K)
    sizes = np.empty(K, dtype=np.int64)
    sizes[ranks] = by_rank
    return _partition_from_sizes(V, sizes, rng.stream_key(rng.SEED_BASE, config, _P_SHUFFLE, seed))


def heavy_tail_partition(V: int, K: int, frac0: float = 0.6, s: float = 1.3, seed: int = 0,
                         config: int = 0) -> Partition:
    """Class 0 holds floor(frac0*V) tokens; the other K-1 classes share the rest ~ rank^-s, each >= 1."""
    assert K >= 2
    n0 = int(np.floor(frac0 * V))
    rest = V - n0
    assert rest >= K - 1
    w = np.arange(1, K, dtype=np.float64) ** (-s)
    sizes = np.empty(K, dtype=np.int64)
    sizes[0] = n0
    sizes[1:] = 1 + _largest_remainder(rest - (K - 1), w)
    return _partition_from_sizes(V, sizes, rng.stream_key(rng.SEED_BASE, config, _P_SHUFFLE, seed))


def identity_partition(V: int) -> Partition:
    """K = V, every token its own class."""
    a = np.arange(V, dtype=np.int32)
    return Partition(V=V, K=V, c=a.copy(), r=a.copy(), sizes=np.ones(V, dtype=np.int64))


def pack_bits(bits: np.ndarray) -> np.ndarray:
    """bool/0-1 array [..., n] -> uint32 [..., ceil(n/32)], bit j of word w = element 32*w + j."""
    bits = np.asarray(bits).astype(np.uint8)
    n = bits.shape[-1]
    nw = (n + 31) // 32
    pad = nw * 32 - n
    if pad:
        bits = np.concatenate([bits, np.zeros(bits.shape[:-1] + (pad,), dtype=np.uint8)], axis=-1)
    by = np.packbits(bits, axis=-1, bitorder="little")
    return np.ascontiguousarray(by).view("<u4").reshape(bits.shape[:-1] + (nw,))


def unpack_bits(words: np.ndarray, n: int) -> np.ndarray:
    """Inverse of :func:`pack_bits` for the first ``n`` elements."""
    w = np.ascontiguousarray(words, dtype="<u4")
    by = w.view(np.uint8).reshape(w.shape[:-1] + (w.shape[-1] * 4,))
    return np.unpackbits(by, axis=-1, bitorder="little")[..., :n].astype(bool)


def class_mask_bernoulli(K: int, B: int, p, key) -> np.ndarray:
    """Each class allowed independently with probability ``p`` (scalar, or one value per row)."""
    p = np.broadcast_to(np.asarray(p, dtype=np.float64).reshape(-1, 1), (B, 1))
    u = rng.uniform(key, B * K).reshape(B, K)
    return pack_bits(u < p)


def class_mask_n_classes(K: int, B: int, nmin: int, nmax: int, key) -> np.ndarray:
    """Each row allows n distinct classes, n uniform in nmin..nmax, classes uniform without replacement."""
    bits = np.zeros((B, K), dtype=bool)
    span = nmax - nmin + 1
    n = nmin + (rng.u64(key, B) % np.uint64(span)).astype(np.int64)
    draws = (rng.u64(key, B * 4 * nmax, offset=B) % np.uint64(K)).astype(np.int64).reshape(B, 4 * nmax)
    for b in range(B):
        _, first = np.unique(draws[b], return_index=True)
        chosen = draws[b][np.sort(first)][: n[b]]
        bits[b, chosen] = True
    return pack_bits(bits)


def logits_normal(B: int, V: int, sigma: float, dtype: str, key_ids, spikes: int = 0,
                  spike_value: float = 8.0) -> np.ndarray:
    """[B, V] logits ~ N(0, sigma^2): float32, or bfloat16 bit patterns (uint16) for dtype 'bf16'.

    ``spikes`` > 0 adds ``spike_value`` at that many distinct uniformly chosen token ids per row.
    """
    out = np.empty((B, V), dtype=np.float32)
    rows_per_block = max(1, (1 << 22) // V)
    for b0 in range(0, B, rows_per_block):
        b1 = min(B, b0 + rows_per_block)
        key = rng.stream_key(*key_ids, _P_LOGITS, b0)
        out[b0:b1] = rng.normal_f32(key, (b1 - b0) * V, sigma).reshape(b1 - b0, V)
    if spikes:
        key = rng.stream_key(*key_ids, _P_SPIKES)
        draws = (rng.u64(key, B * 2 * spikes) % np.uint64(V)).astype(np.int64).reshape(B, 2 * spikes)
        for b in range(B):
            _, first = np.unique(draws[b], return_index=True)
            ids = draws[b][np.sort(first)][:spikes]
            out[b, ids] += np.float32(spike_value)
    if dtype == "bf16":
        return rng.f32_to_bf16_bits(out.reshape(-1)).reshape(B, V)
    assert dtype == "f32"
    return out


# The five workloads. "steps" is the number of decode steps the full-size parity run covers.
CONFIGS: Dict[int, dict] = {
    1: dict(name="tiny", V=32000, K=256, B=1, dtype="f32", sigma=1.0, steps=100, zipf_s=1.1,
            mask=("bernoulli", 0.3), n_partitions=1),
    2: dict(name="llama3-size", V=128256, K=2048, B=32, dtype="bf16", sigma=2.0, steps=1000, zipf_s=1.1,
            mask=("bernoulli", 0.1), n_partitions=1),
    3: dict(name="qwen-size", V=151936, K=4096, B=128, dtype="f32", sigma=1.0, steps=500, zipf_s=1.1,
            mask=("round_robin", (0.01, 0.1, 0.5, 0.99)), n_partitions=1, spikes=50),
    4: dict(name="heavy-tail", V=256000, K=16384, B=256, dtype="bf16", sigma=1.0, steps=200, zipf_s=1.3,
            mask=("row_uniform", None), n_partitions=8, heavy=0.6),
    5: dict(name="sparse-stress", V=128256, K=512, B=1024, dtype="f32", sigma=1.0, steps=200, zipf_s=1.1,
            mask=("n_classes", (1, 5)), n_partitions=1),
}


@dataclass
class Workload:
    """One of the five workloads, optionally shrunk (fewer rows / smaller V, K) for quick parity runs."""

    config: int
    V: int
    K: int
    B: int
    dtype: str
    partitions: List[Partition]
    row_part: Optional[np.ndarray]  # int32 [B] or None (all rows use partition 0)
    spec: dict = field(repr=False, default_factory=dict)

    def class_masks(self, step: int) -> np.ndarray:
        """uint32 [B, ceil(K/32)] for decode step ``step``."""
        kind, arg = self.spec["mask"]
        key = rng.stream_key(rng.SEED_BASE, self.config, _P_MASK, step)
        if kind == "bernoulli":
            return class_mask_bernoulli(self.K, self.B, arg, key)
        if kind == "round_robin":
            p = np.array([arg[b % len(arg)] for b in range(self.B)])
            return class_mask_bernoulli(self.K, self.B, p, key)
        if kind == "row_uniform":
            p = rng.uniform(rng.stream_key(rng.SEED_BASE, self.config, _P_DENSITY), self.B)
            return class_mask_bernoulli(self.K, self.B, p, key)
        if kind == "n_classes":
            return class_mask_n_classes(self.K, self.B, arg[0], arg[1],
                                        rng.stream_key(rng.SEED_BASE, self.config, _P_NCLS, step))
        raise ValueError(kind)

    def logits(self, step: int) -> np.ndarray:
        """Fresh [B, V] logits for decode step ``step`` (float32, or uint16 bf16 bit patterns)."""
        return logits_normal(self.B, self.V, self.spec["sigma"], self.dtype,
                             (rng.SEED_BASE, self.config, step), spikes=self.spec.get("spikes", 0))

    def uniforms(self, step: int) -> np.ndarray:
        """float32 [B] in [0, 1): the one random number per row that a sampling step consumes."""
        key = rng.stream_key(rng.SEED_BASE, self.config, _P_UNIFORM, step)
        u = (rng.u64(key, self.B) >> np.uint64(40)).astype(np.float32) * np.float32(2.0 ** -24)  # 24 bits: exact in float32
        return u

    def partition_of_row(self, b: int) -> Partition:
        return self.partitions[0 if self.row_part is None else int(self.row_part[b])]


def make_workload(config: int, B: Optional[int] = None, V: Optional[int] = None,
                  K: Optional[int] = None) -> Workload:
    """Build workload ``config`` (1..5); B, V, K override the full sizes for reduced parity cases."""
    spec = dict(CONFIGS[config])
    V = int(V or spec["V"])
    K = int(K or spec["K"])
    B = int(B or spec["B"])
    parts = []
    for p in range(spec["n_partitions"]):
        if "heavy" in spec:
            parts.append(heavy_tail_partition(V, K, spec["heavy"], spec["zipf_s"], seed=p, config=config))
        else:
            parts.append(zipf_partition(V, K, spec["zipf_s"], seed=p, config=config))
    row_part = None
    if spec["n_partitions"] > 1:
        row_part = (np.arange(B) % spec["n_partitions"]).astype(np.int32)
    return Workload(config=config, V=V, K=K, B=B, dtype=spec["dtype"], partitions=parts,
                    row_part=row_part, spec=spec)
