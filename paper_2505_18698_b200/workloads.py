"""Seeded synthetic inputs and the five benchmark configurations.

This module holds no arithmetic of the method: it only draws Q, K, V.  Both the
CUDA path's tests/benchmark and the CPU oracle's tests take their inputs from
here, so the two sides see bit-identical tensors.

Recipe (the paper benchmarks on random Q, K, V; Sec. 4 'Benchmarking'):
    W[h]  : (r, d)   rank-r basis per head, shared by Q and K and across the batch
    CQ,CK : (batch, heads, N, r) independent coefficients
    GQ,GK,GV : (batch, heads, N, d) i.i.d. N(0,1)
    Q = GQ + s * (CQ @ W[h]) / sqrt(r),   K = GK + s * (CK @ W[h]) / sqrt(r),   V = GV
then rounded (round-to-nearest-even) to the configuration's dtype.  The rank-r
component stands in for the peaky, structured attention of trained encoders.
All draws come from numpy's Philox generator in float32, in the order
W, CQ, CK, GQ, GK, GV.
"""
from __future__ import annotations

from dataclasses import dataclass, asdict

import numpy as np

DTYPE_CODES = {"f32": 0, "f16": 1, "bf16": 2}
DTYPE_BYTES = {"f32": 4, "f16": 2, "bf16": 2}


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    heads: int
    N: int
    d: int
    b: int
    T: int
    dtype: str          # "f32" | "f16" | "bf16"
    rank: int           # r (0 = pure i.i.d. N(0,1))
    s: float            # scale of the shared rank-r component
    seed: int
    note: str = ""

    @property
    def m(self) -> int:
        return self.N // self.b

    @property
    def BH(self) -> int:
        return self.batch * self.heads

    @property
    def tokens(self) -> int:
        return self.batch * self.N

    def algorithmic_bytes(self) -> int:
        """One read of Q, K, V and one write of Y (Sec. 3: Theta(N d) IO)."""
        return 4 * self.BH * self.N * self.d * DTYPE_BYTES[self.dtype]

    def algorithmic_flops(self) -> int:
        """2 x the multiply-accumulate count the paper's tables use:
        MACs/head = T*2*N*d*(b+m) + N*b*d  (reproduces Tab. 1 and Tab. 2)."""
        return 2 * self.BH * macs_per_head(self.N, self.d, self.b, self.T)

    def exps(self) -> int:
        return self.BH * self.T * self.N * (self.b + self.m)

    def as_dict(self):
        return asdict(self)


def macs_per_head(N: int, d: int, b: int, T: int) -> int:
    """Multiply-accumulates of one head: per step four contractions of
    N*b*d or N*m*d each (Eq. 7-10), plus y = R*Vb (N*b*d); the final
    L*y contraction replaces the last step's alpha_R update."""
    m = N // b
    return T * 2 * N * d * (b + m) + N * b * d


WORKLOADS = {
    "C1": Workload("C1", 1, 1, 256, 64, 16, 1, "f32", 0, 0.0, 0,
                   "single-head tiny, i.i.d. N(0,1)"),
    "C2": Workload("C2", 64, 12, 256, 64, 16, 1, "f16", 8, 2.0, 1,
                   "ViT-B-like encoder attention"),
    "C3": Workload("C3", 16, 12, 1024, 64, 32, 2, "bf16", 8, 2.0, 2,
                   "RoBERTa-base-like"),
    "C4": Workload("C4", 4, 16, 4096, 64, 64, 2, "bf16", 16, 1.5, 3,
                   "medium sequence"),
    "C5": Workload("C5", 1, 16, 16384, 64, 128, 2, "bf16", 16, 1.5, 4,
                   "long sequence"),
}

# Shapes of the paper's short-sequence experiments (Sec. 5) with blocks that are not 16 x 16:
# selectable in bench.py by name, not part of the configuration list the bench reports on.
EXTRA_WORKLOADS = {
    "S1": Workload("S1", 64, 12, 210, 64, 14, 2, "f16", 8, 1.0, 5,
                   "ViT-B sequence (197 padded to 15 blocks of 14), two rounds"),
    "S2": Workload("S2", 32, 12, 384, 64, 24, 1, "f16", 8, 1.0, 6,
                   "RoBERTa sequence 384 as 16 blocks of 24, one round"),
    "S3": Workload("S3", 2, 16, 8192, 64, 64, 1, "bf16", 8, 1.0, 7,
                   "BART sequence 8192 as 128 blocks of 64 (m != b), one round"),
    "S4": Workload("S4", 1, 8, 7680, 48, 128, 2, "f16", 8, 1.0, 8,
                   "graph transformer: 7600 nodes padded to 60 blocks of 128, d = 48, two rounds"),
    "S5": Workload("S5", 8, 16, 256, 72, 16, 3, "f16", 8, 1.0, 9,
                   "DiT: 256 image tokens as 16 blocks of 16, d = 72, three rounds"),
    "S6": Workload("S6", 32, 12, 384, 64, 48, 1, "f16", 8, 1.0, 10,
                   "RoBERTa sequence 384 as 8 blocks of 48, one round"),
}


# --------------------------------------------------------------------------- rounding
def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float32 array to `dtype` (RNE) and return it as float32 again."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "f32":
        return x
    if dtype == "f16":
        return x.astype(np.float16).astype(np.float32)
    if dtype == "bf16":
        u = x.view(np.uint32).astype(np.uint64)
        u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
        return u.astype(np.uint32).view(np.float32).reshape(x.shape)
    raise ValueError(dtype)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 values that are exactly bf16-representable -> uint16 bit patterns."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


def from_bf16_bits(u: np.ndarray) -> np.ndarray:
    return (u.astype(np.uint32) << 16).view(np.float32)


# --------------------------------------------------------------------------- generator
def make_qkv(batch, heads, N, d, dtype="f32", rank=0, s=0.0, seed=0, head_slice=None):
    """Returns (Q, K, V) as float32 arrays of shape (batch, heads, N, d) whose
    values are exactly representable in `dtype`."""
    rng = np.random.Generator(np.random.Philox(seed))
    f32 = np.float32
    if rank > 0:
        W = rng.standard_normal((heads, rank, d), dtype=f32)
        CQ = rng.standard_normal((batch, heads, N, rank), dtype=f32)
        CK = rng.standard_normal((batch, heads, N, rank), dtype=f32)
    GQ = rng.standard_normal((batch, heads, N, d), dtype=f32)
    GK = rng.standard_normal((batch, heads, N, d), dtype=f32)
    GV = rng.standard_normal((batch, heads, N, d), dtype=f32)
    if rank > 0:
        c = f32(s / np.sqrt(rank))
        GQ += c * np.einsum("ehnr,hrd->ehnd", CQ, W)
        GK += c * np.einsum("ehnr,hrd->ehnd", CK, W)
    return (round_to_dtype(GQ, dtype), round_to_dtype(GK, dtype), round_to_dtype(GV, dtype))


def make_workload_inputs(w: Workload):
    return make_qkv(w.batch, w.heads, w.N, w.d, w.dtype, w.rank, w.s, w.seed)


def shard_units(total_units: int, world_size: int, rank: int):
    """Contiguous slice [lo, hi) of the batch*heads units owned by `rank`.
    Heads are independent (every equation of the paper is per head), so the
    multi-GPU path is a partition with no data-path collective."""
    base, rem = divmod(total_units, world_size)
    lo = rank * base + min(rank, rem)
    hi = lo + base + (1 if rank < rem else 0)
    return lo, hi
