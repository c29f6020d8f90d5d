"""Seeded synthetic workloads shared by the tests, the smoke check and the benchmark.

This module holds no attention arithmetic and no chunking logic: only random lengths, random
values and bf16 bit handling.  The private long-context datasets the paper trains on
(Section 6.1) are not available; these length mixes take the shape the paper states for them
(Section 2.2: lengths spread over four orders of magnitude, most sequences short, a thin tail up
to 256K; Section 6.1: per-rank token budgets of 4K at 32K context and 8K at 256K context, times an
inner Ulysses group of 8) and stand in for them.

Values are bf16 N(0,1), generated per (tensor, head) from independent streams so that a subset of
heads can be produced without materialising the rest.
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field
from typing import Dict, List, Sequence

import numpy as np

D_QK = 192
D_V = 128
SEED = 34318
TENSOR_ID = {"q": 0, "k": 1, "v": 2, "do": 3}


# ------------------------------------------------------------------------------------------------
# bf16 bit handling (round-to-nearest-even, the conversion a GPU cast performs)
# ------------------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    nan = np.isnan(x)
    rounded = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    out = rounded.astype(np.uint16)
    if nan.any():
        out[nan] = np.uint16(0x7FC0)
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# ------------------------------------------------------------------------------------------------
# length lists
# ------------------------------------------------------------------------------------------------
def _fill(draw, total: int, l_min: int) -> List[int]:
    """Draw lengths until `total` tokens are filled; the last sequence absorbs a short tail."""
    out: List[int] = []
    remaining = total
    while remaining > 0:
        length = min(int(draw()), remaining)
        if remaining - length < l_min:
            length = remaining
        out.append(length)
        remaining -= length
    return out


def lengths_lognormal(total: int = 32768, median: int = 1024, sigma: float = 1.0, lo: int = 64,
                      hi: int = 32768, seed: int = SEED) -> List[int]:
    rng = np.random.Generator(np.random.PCG64(seed))
    return _fill(lambda: np.clip(np.round(np.exp(rng.normal(np.log(median), sigma))), lo, hi),
                 total, lo)


def lengths_skewed(long_len: int = 98304, rest: int = 32768, alpha: float = 1.2, lo: int = 256,
                   hi: int = 32768, seed: int = SEED) -> List[int]:
    rng = np.random.Generator(np.random.PCG64(seed))
    tail = _fill(lambda: np.clip(np.floor(lo * (1.0 + rng.pareto(alpha))), lo, hi), rest, lo)
    seqs = np.array([long_len] + tail, dtype=np.int64)
    perm = np.random.Generator(np.random.PCG64(seed + 1)).permutation(len(seqs))
    return [int(x) for x in seqs[perm]]


def lengths_uniform(total: int = 65536, lo: int = 64, hi: int = 512, seed: int = SEED) -> List[int]:
    rng = np.random.Generator(np.random.PCG64(seed))
    return _fill(lambda: rng.integers(lo, hi + 1), total, lo)


def lengths_sha1(lengths: Sequence[int]) -> str:
    return hashlib.sha1(np.asarray(lengths, dtype=np.int32).tobytes()).hexdigest()


def cu_seqlens(lengths: Sequence[int]) -> np.ndarray:
    cu = np.zeros(len(lengths) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(np.asarray(lengths, dtype=np.int64))
    return cu


# ------------------------------------------------------------------------------------------------
# values
# ------------------------------------------------------------------------------------------------
def tensor_bits(name: str, total: int, heads: Sequence[int], n_heads_total: int | None = None,
                seed: int = SEED) -> np.ndarray:
    """bf16 N(0,1) bits of tensor `name` for the listed heads, shape [T, len(heads), d]."""
    del n_heads_total
    d = D_V if name in ("v", "do") else D_QK
    out = np.empty((total, len(heads), d), dtype=np.uint16)
    for slot, head in enumerate(heads):
        rng = np.random.default_rng([seed, TENSOR_ID[name], int(head)])
        out[:, slot, :] = f32_to_bf16_bits(rng.standard_normal((total, d), dtype=np.float32))
    return out


# ------------------------------------------------------------------------------------------------
# the five configurations
# ------------------------------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    lengths: List[int]
    n_heads: int
    cp_r: int = 0                 # outer-ring degree used to cut every sequence (0 = not cut);
                                  # 1 cuts a sequence in two chunks (floor(L/2), rest)
    causal: bool = True
    note: str = ""
    extra: Dict[str, object] = field(default_factory=dict)

    @property
    def total(self) -> int:
        return int(sum(self.lengths))

    @property
    def scale(self) -> np.float32:
        return np.float32(1.0 / np.sqrt(np.float32(D_QK)))

    @property
    def causal_pairs_total(self) -> int:
        return int(sum(l * (l + 1) // 2 for l in self.lengths))

    def flops_fwd(self) -> float:
        """Causal-pair convention: 2 * pairs * h * (d_qk + d_v); the backward counts 2.5x."""
        return 2.0 * self.causal_pairs_total * self.n_heads * (D_QK + D_V)

    def cu(self) -> np.ndarray:
        return cu_seqlens(self.lengths)

    def tensors(self, heads: Sequence[int] | None = None, names=("q", "k", "v", "do")):
        heads = list(range(self.n_heads)) if heads is None else list(heads)
        return {n: tensor_bits(n, self.total, heads) for n in names}


def workload(name: str) -> Workload:
    if name == "tiny":
        return Workload("tiny", [7, 33, 128, 300], 4,
                        note="4 packed sequences, one pair per sequence")
    if name == "tiny_split":
        return Workload("tiny_split", [300], 4, cp_r=1,
                        note="the 300-token sequence cut into 2 chunks (3 pairs), merged")
    if name == "packed32k":
        return Workload("packed32k", lengths_lognormal(), 16,
                        note="32K-token packed microbatch, log-normal lengths (median 1K, sigma 1)")
    if name == "ring256k":
        return Workload("ring256k", [262144], 16, cp_r=4,
                        note="one 256K sequence, outer ring of 4: 8 zigzag chunks, 36 pairs, merged")
    if name == "ring64k":
        return Workload("ring64k", [65536], 16, cp_r=1,
                        note="a slice of the 256K configuration for profiling: one 64K sequence in two of its "
                             "32K-token chunks, 2 diagonal pairs and 1 full pair, merged")
    if name == "skewed128k":
        return Workload("skewed128k", lengths_skewed(), 16,
                        note="one 96K sequence + Pareto(1.2) tail filling 32K")
    if name == "short64k":
        return Workload("short64k", lengths_uniform(), 32,
                        note="64K tokens of sequences with lengths uniform in [64, 512]")
    if name == "short64k_split":
        return Workload("short64k_split", lengths_uniform(), 32, cp_r=1,
                        note="many-short with every sequence cut in two chunks and merged")
    raise KeyError(name)


WORKLOADS = ("tiny", "tiny_split", "packed32k", "ring256k", "ring64k", "skewed128k", "short64k",
             "short64k_split")
