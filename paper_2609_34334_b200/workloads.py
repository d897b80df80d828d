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


_BLOCK = 1 << 17   # elements per generation block: temporaries stay cache resident


def _blocked(fn, n: int, start: int) -> np.ndarray:
    """Evaluates fn(first_index, length) -> float32 block over [start, start+n) block by block."""
    out = np.empty(n, dtype=np.float32)
    for lo in range(0, n, _BLOCK):
        m = min(_BLOCK, n - lo)
        out[lo:lo + m] = fn(start + lo, m)
    return out


def uniform(seed: int, rank: int, n: int, dtype: str, start: int = 0) -> np.ndarray:
    """uniform[-1, 1): k / 2^23 - 1 with k the top 24 bits of the word (exact in fp32)."""
    def block(first, m):
        k = (raw_bits(seed, rank, 0, first, m) >> np.uint64(40)).astype(np.float32)
        return k * np.float32(2.0 ** -23) - np.float32(1.0)

    return _finish(_blocked(block, n, start), dtype)


def normal(seed: int, rank: int, n: int, dtype: str, sigma: float = 1.0, start: int = 0) -> np.ndarray:
    """normal(0, sigma) by Box-Muller in float64, then cast to float32 (and bf16 if asked)."""
    def block(first, m):
        u1 = ((raw_bits(seed, rank, 1, first, m) >> np.uint64(11)).astype(np.float64) + 0.5) * 2.0 ** -53
        u2 = ((raw_bits(seed, rank, 2, first, m) >> np.uint64(11)).astype(np.float64) + 0.5) * 2.0 ** -53
        z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
        return (z * sigma).astype(np.float32)

    return _finish(_blocked(block, n, start), dtype)


def small_integers(seed: int, rank: int, n: int, dtype: str, bound: int = 8, start: int = 0) -> np.ndarray:
    """integers in [-bound, bound]; every partial sum over up to 8 ranks is exact in bf16 and fp32."""
    def block(first, m):
        k = (raw_bits(seed, rank, 3, first, m) >> np.uint64(33)) % np.uint64(2 * bound + 1)
        return k.astype(np.float32) - np.float32(bound)

    return _finish(_blocked(block, n, start), dtype)


# ---- position-dependent inputs that can also be produced ON THE DEVICE (full-size parity runs) --------------------
# A 32-bit integer hash of (seed, rank, element index) written with 64-bit integer operations that never overflow, so
# numpy (host windows for the oracle) and torch (whole buffers, generated where they are used) give the same values.
_H_A, _H_B, _H_C, _H_M1, _H_M2 = 2654435761, 0x9E3779B1, 0x85EBCA6B, 0x7FEB352D, 0x2C1B3C6D


def _hash32(xp, idx, seed: int, rank: int):
    """idx: int64 array/tensor of element indices below 2^31.  Returns int64 values in [0, 2^32)."""
    m = 0xFFFFFFFF
    h = (idx * _H_A + ((rank + 1) * _H_B + (seed + 1) * _H_C) % (1 << 32)) & m
    h = h ^ (h >> 16)
    h = (h * _H_M1) & m
    h = h ^ (h >> 15)
    h = (h * _H_M2) & m
    return h ^ (h >> 16)


def hashed(kind: str, seed: int, rank: int, start: int, n: int, dtype: str) -> np.ndarray:
    """Elements start..start+n-1 of rank `rank`: kind "int" = integers in [-8, 8] (every partial sum over up to 8 ranks is
    exact in bf16 and fp32, so the all-reduce result is the exact integer sum whatever the order), kind "uniform" =
    k / 2^23 - 1 with k the top 24 bits of the hash.  No period: the value depends on the element's position."""
    h = _hash32(np, np.arange(start, start + n, dtype=np.int64), seed, rank)
    if kind == "int":
        x = (h % 17 - 8).astype(np.float32)
    elif kind == "uniform":
        x = (h >> 8).astype(np.float32) * np.float32(2.0 ** -23) - np.float32(1.0)
    else:
        raise ValueError(kind)
    return _finish(x, dtype)


def hashed_device(kind: str, seed: int, rank: int, n: int, dtype: str, device="cuda", block: int = 1 << 25):
    """The same values as hashed(kind, seed, rank, 0, n, dtype) as a torch tensor on `device` (float32, or bfloat16 for
    "bf16"), generated block by block so that the 64-bit temporaries stay small."""
    import torch

    out = torch.empty(n, dtype=torch.float32 if dtype == "fp32" else torch.bfloat16, device=device)
    for lo in range(0, n, block):
        m = min(block, n - lo)
        h = _hash32(torch, torch.arange(lo, lo + m, dtype=torch.int64, device=device), seed, rank)
        if kind == "int":
            x = (h % 17 - 8).to(torch.float32)
        elif kind == "uniform":
            x = (h >> 8).to(torch.float32) * (2.0 ** -23) - 1.0
        else:
            raise ValueError(kind)
        out[lo:lo + m] = x.to(out.dtype)      # float32 -> bfloat16 rounds to nearest even, as _finish does
    return out


def _finish(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "fp32":
        return np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "bf16":
        return _to_bf16_bits(x)
    raise ValueError("dtype must be 'fp32' or 'bf16'")


def elem_size(dtype: str) -> int:
    return {"fp32": 4, "bf16": 2}[dtype]


def rank_inputs(dist: str, seed: int, R: int, n: int, dtype: str, sigma: float = 1.0):
    """R per-rank arrays of n elements (large requests are generated by one thread per rank)."""
    if dist == "uniform":
        fn = lambda r: uniform(seed, r, n, dtype)
    elif dist == "normal":
        fn = lambda r: normal(seed, r, n, dtype, sigma)
    elif dist == "int":
        fn = lambda r: small_integers(seed, r, n, dtype)
    else:
        raise ValueError(dist)
    if R * n >= (1 << 22) and R > 1:
        from concurrent.futures import ThreadPoolExecutor

        with ThreadPoolExecutor(max_workers=min(R, 8)) as pool:
            return list(pool.map(fn, range(R)))
    return [fn(r) for r in range(R)]


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


def gradient_bucket(g: GradientStream, b: int):
    """The R per-rank arrays of bucket b of the gradient stream: elements [b * per, b * per + len) of every rank's flat
    gradient, normal(0, sigma) from the stream's seed (position independent, so any bucket can be produced alone)."""
    sizes = g.buckets()
    per = sizes[0]
    n = sizes[b]
    from concurrent.futures import ThreadPoolExecutor

    with ThreadPoolExecutor(max_workers=min(g.R, 8)) as pool:
        return list(pool.map(lambda r: normal(g.seed, r, n, g.dtype, g.sigma, start=b * per), range(g.R)))


@dataclass(frozen=True)
class Sweep:
    name: str = "c5_size_sweep"
    sizes: tuple = field(default_factory=lambda: tuple(1 << k for k in range(12, 31)))   # 4 KiB .. 1 GiB per rank
    ranks: tuple = (2, 4, 8)
    dtypes: tuple = ("fp32", "bf16")
    ops: tuple = ("allreduce", "reduce_scatter", "allgather", "sendrecv")
    seed: int = 4


C5_SWEEP = Sweep()
