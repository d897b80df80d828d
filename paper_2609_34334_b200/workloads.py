"""Seeded synthetic inputs and workload shapes.

This module holds NO arithmetic of the collectives: it only produces the per-rank input arrays that
both the CUDA path and the CPU oracle consume, plus the shapes of the benchmark workloads.

Generator: counter based (splitmix64 keyed by seed, rank and element index), so any slice of any
rank's buffer can be produced independently and in any order.  fp32 values are numpy float32; bf16
values are returned as uint16 bit patterns (float32 rounded to nearest-even by torch's CPU cast).

The workloads stand in for the paper's: nccl-tests style sweeps from small messages to 1 GiB
(Sec. 5 "Communication benchmarks") and GPT-6.7B bf16 traffic at sequence length 2048 (Table 2,
"End-to-end workloads"): data-parallel gradient buckets and pipeline-parallel activations.
Contents are seeded random numbers; moves are data independent and only the sums look at values.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = z + _GOLD
        z = (z ^ (z >> np.uint64(30))) * _C1
        z = (z ^ (z >> np.uint64(27))) * _C2
        return z ^ (z >> np.uint64(31))


def raw_bits(seed: int, rank: int, lane: int, start: int, n: int) -> np.ndarray:
    """n 64-bit words for elements start..start+n-1 of (seed, rank, lane)."""
    key = _mix(np.array([(seed & 0xFFFFFFFF) << 32 | (rank & 0xFFFFFF) << 8 | (lane & 0xFF)], dtype=np.uint64))[0]
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + n, dtype=np.uint64)
        return _mix(key + idx * _GOLD)


def _to_bf16_bits(f32: np.ndarray) -> np.ndarray:
    import torch

    t = torch.from_numpy(np.ascontiguousarray(f32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def uniform(seed: int, rank: int, n: int, dtype: str, start: int = 0) -> np.ndarray:
    """uniform[-1, 1): k / 2^23 - 1 with k the top 24 bits of the word (exact in fp32)."""
    k = (raw_bits(seed, rank, 0, start, n) >> np.uint64(40)).astype(np.float32)
    x = k * np.float32(2.0 ** -23) - np.float32(1.0)
    return _finish(x, dtype)


def normal(seed: int, rank: int, n: int, dtype: str, sigma: float = 1.0, start: int = 0) -> np.ndarray:
    """normal(0, sigma) by Box-Muller in float64, then cast to float32 (and bf16 if asked)."""
    u1 = ((raw_bits(seed, rank, 1, start, n) >> np.uint64(11)).astype(np.float64) + 0.5) * 2.0 ** -53
    u2 = ((raw_bits(seed, rank, 2, start, n) >> np.uint64(11)).astype(np.float64) + 0.5) * 2.0 ** -53
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return _finish((z * sigma).astype(np.float32), dtype)


def small_integers(seed: int, rank: int, n: int, dtype: str, bound: int = 8, start: int = 0) -> np.ndarray:
    """integers in [-bound, bound]; every partial sum over up to 8 ranks is exact in bf16 and fp32."""
    k = (raw_bits(seed, rank, 3, start, n) >> np.uint64(33)) % np.uint64(2 * bound + 1)
    return _finish(k.astype(np.float32) - np.float32(bound), dtype)


def _finish(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "fp32":
        return np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "bf16":
        return _to_bf16_bits(x)
    raise ValueError("dtype must be 'fp32' or 'bf16'")


def elem_size(dtype: str) -> int:
    return {"fp32": 4, "bf16": 2}[dtype]


def rank_inputs(dist: str, seed: int, R: int, n: int, dtype: str, sigma: float = 1.0):
    """R per-rank arrays of n elements."""
    if dist == "uniform":
        return [uniform(seed, r, n, dtype) for r in range(R)]
    if dist == "normal":
        return [normal(seed, r, n, dtype, sigma) for r in range(R)]
    if dist == "int":
        return [small_integers(seed, r, n, dtype) for r in range(R)]
    raise ValueError(dist)


# ----------------------------------------------------------------------------------------------
# Workload shapes (the five benchmark configurations)
# ----------------------------------------------------------------------------------------------
@dataclass(frozen=True)
class Collective:
    name: str
    op: str            # "allreduce" | "reduce_scatter+allgather" | "allgather" | "sendrecv"
    R: int
    count: int         # elements per rank buffer (allreduce convention: size of each X_r)
    dtype: str
    dist: str
    seed: int
    sigma: float = 1.0
    note: str = ""

    @property
    def bytes_per_rank(self) -> int:
        return self.count * elem_size(self.dtype)


C1_SMALL_ALLREDUCE = Collective("c1_allreduce_r4_fp32_4MiB", "allreduce", 4, 1_048_576, "fp32", "uniform", 0,
                                note="R=4, 1,048,576 fp32 per rank, uniform[-1,1), 4 ring chunks")
C2_DP_BUCKET = Collective("c2_dp_bucket_r8_bf16_25MiB", "reduce_scatter+allgather", 8, 13_107_200, "bf16", "normal", 1,
                          sigma=1e-3, note="R=8, 25 MiB bf16 gradient bucket per rank, normal(0,1e-3), 8 ring chunks")


@dataclass(frozen=True)
class Pipeline:
    """Pipeline-parallel point-to-point wave: microbatch m travels stage 0 -> 1 -> ... -> stages-1."""
    name: str = "c3_pp_sendrecv_8stages_16mb_64MiB"
    stages: int = 8
    microbatches: int = 16
    shape: tuple = (4, 2048, 4096)   # microbatch x seq x hidden
    dtype: str = "bf16"
    seed: int = 2
    gemm_probe: tuple = (4096, 4096, 4096)

    @property
    def count(self) -> int:
        return int(np.prod(self.shape))

    @property
    def hops(self) -> int:
        return (self.stages - 1) * self.microbatches


C3_PIPELINE = Pipeline()


@dataclass(frozen=True)
class GradientStream:
    """GPT-6.7B shaped data-parallel gradients cut into fixed-size buckets."""
    name: str = "c4_gpt6p7b_dp_allreduce_r8_bf16_40MiB_buckets"
    R: int = 8
    layers: int = 32
    hidden: int = 4096
    ffn: int = 16384
    dtype: str = "bf16"
    sigma: float = 1e-3
    seed: int = 3
    bucket_bytes: int = 40 << 20
    gemm_probe: tuple = (8192, 4096, 16384)

    @property
    def elements_per_layer(self) -> int:
        h, f = self.hidden, self.ffn
        return 3 * h * h + h * h + h * f + f * h   # qkv, proj, fc1, fc2 weights

    @property
    def total_elements(self) -> int:
        return self.layers * self.elements_per_layer

    def buckets(self):
        """List of bucket sizes in elements (full buckets, then one ragged tail)."""
        per = self.bucket_bytes // elem_size(self.dtype)
        full, rest = divmod(self.total_elements, per)
        return [per] * full + ([rest] if rest else [])


C4_GRADIENTS = GradientStream()


@dataclass(frozen=True)
class Sweep:
    name: str = "c5_size_sweep"
    sizes: tuple = field(default_factory=lambda: tuple(1 << k for k in range(12, 31)))   # 4 KiB .. 1 GiB per rank
    ranks: tuple = (2, 4, 8)
    dtypes: tuple = ("fp32", "bf16")
    ops: tuple = ("allreduce", "reduce_scatter", "allgather", "sendrecv")
    seed: int = 4


C5_SWEEP = Sweep()
