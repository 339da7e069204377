"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random tensors (numpy, host side).  It holds none of the
method's arithmetic: no features, no fits, no attention.  Both the CUDA path
and the CPU checker are fed from these arrays, so neither depends on the other.

The five workloads mirror the benchmark configurations:
  cfg1  tiny bidirectional SDERF, fp32: B1 H1 L256 d16 dv16 M32, iid Gaussian Omega
  cfg2  bidirectional SDERF, bf16: B8 H8 L4096 d64 dv64 M256, orthogonal Omega,
        per-head mean shift N(0, 0.1^2) on Q and on K
  cfg3  causal ADERF, bf16: B4 H12 L8192 d64 dv64 M256, chunk 128
  cfg4  2^20 (x, y) pairs, d64, M64: Uniform[0,1] entries, L2-normalised, times 2
  cfg5  causal SDERF, bf16: B1 H16 L65536 d128 dv128 M512, chunk 256,
        5% of token positions scaled by 3
Q and K entries are N(0,1)/d^(1/4), so they already are the x and y of the
method (qk_scale = 1); V entries are N(0,1).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    L: int
    d: int
    dv: int
    M: int
    dtype: str            # "f32" or "bf16"
    variant: str          # "sderf", "aderf", ...
    causal: bool
    chunk: int
    omega: str            # "iid" or "orthogonal"
    head_shift_std: float = 0.0
    outlier_frac: float = 0.0
    outlier_scale: float = 1.0
    seed: int = 0

    def scaled(self, **kw) -> "Workload":
        """A smaller (or otherwise modified) case of the same recipe."""
        return replace(self, **kw)


WORKLOADS = {
    "cfg1": Workload("cfg1", 1, 1, 256, 16, 16, 32, "f32", "sderf", False, 0, "iid", seed=1000),
    "cfg2": Workload("cfg2", 8, 8, 4096, 64, 64, 256, "bf16", "sderf", False, 0, "orthogonal",
                     head_shift_std=0.1, seed=2000),
    "cfg3": Workload("cfg3", 4, 12, 8192, 64, 64, 256, "bf16", "aderf", True, 128, "orthogonal",
                     seed=3000),
    "cfg3b": Workload("cfg3b", 4, 12, 8192, 64, 64, 256, "bf16", "aderf", False, 0, "orthogonal",
                      seed=3000),
    "cfg5": Workload("cfg5", 1, 16, 65536, 128, 128, 512, "bf16", "sderf", True, 256, "orthogonal",
                     outlier_frac=0.05, outlier_scale=3.0, seed=5000),
    # cfg5 at a quarter of its length: small enough for a profiler capture, inputs still larger than L2
    "cfg5m": Workload("cfg5m", 1, 16, 16384, 128, 128, 512, "bf16", "sderf", True, 256, "orthogonal",
                      outlier_frac=0.05, outlier_scale=3.0, seed=5000),
    # cfg5's few, long sequences (1 x 16 heads x 65536 tokens, x3 outlier tokens) at the head size of cfg2 / cfg3
    "cfg5s": Workload("cfg5s", 1, 16, 65536, 64, 64, 256, "bf16", "sderf", True, 128, "orthogonal",
                      outlier_frac=0.05, outlier_scale=3.0, seed=5500),
}


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bfloat16 (ties to even); result stays float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    u = (u + r) & np.uint32(0xFFFF0000)
    return u.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The uint16 bit patterns of bf16_round(x)."""
    return (bf16_round(x).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def iid_omega(M: int, d: int, seed: int) -> np.ndarray:
    """M rows drawn iid from N(0, I_d)."""
    return _rng(seed, 7).standard_normal((M, d), dtype=np.float32)


def orthogonal_omega(M: int, d: int, seed: int) -> np.ndarray:
    """Block-orthogonal Gaussian directions: ceil(M/d) independent d x d Gaussian
    blocks, each orthogonalised by QR (column signs fixed by the sign of diag R so
    the factor is Haar distributed), each row then rescaled by the norm of an
    independent N(0, I_d) vector (chi-distributed with d degrees of freedom)."""
    rng = _rng(seed, 8)
    blocks = []
    for _ in range(-(-M // d)):
        G = rng.standard_normal((d, d))
        Qm, R = np.linalg.qr(G)
        Qm = Qm * np.sign(np.diag(R))[None, :]
        norms = np.linalg.norm(rng.standard_normal((d, d)), axis=1)
        blocks.append(Qm * norms[:, None])
    return np.concatenate(blocks, axis=0)[:M].astype(np.float32)


def make_omega(w: Workload) -> np.ndarray:
    if w.omega == "iid":
        return iid_omega(w.M, w.d, w.seed)
    return orthogonal_omega(w.M, w.d, w.seed)


def make_qkv(w: Workload):
    """Q, K (B,H,L,d) and V (B,H,L,dv) as float32 arrays; for bf16 workloads the
    values are already rounded to bfloat16, so every consumer sees the same numbers."""
    scale = np.float32(w.d ** -0.25)
    Q = _rng(w.seed, 1).standard_normal((w.B, w.H, w.L, w.d), dtype=np.float32) * scale
    K = _rng(w.seed, 2).standard_normal((w.B, w.H, w.L, w.d), dtype=np.float32) * scale
    V = _rng(w.seed, 3).standard_normal((w.B, w.H, w.L, w.dv), dtype=np.float32)
    if w.head_shift_std > 0.0:
        r = _rng(w.seed, 4)
        mq = r.standard_normal((1, w.H, 1, w.d), dtype=np.float32) * np.float32(w.head_shift_std)
        mk = r.standard_normal((1, w.H, 1, w.d), dtype=np.float32) * np.float32(w.head_shift_std)
        Q += mq
        K += mk
    if w.outlier_frac > 0.0:
        mask = _rng(w.seed, 5).random((w.B, 1, w.L, 1)) < w.outlier_frac
        f = np.where(mask, np.float32(w.outlier_scale), np.float32(1.0)).astype(np.float32)
        Q *= f
        K *= f
    if w.dtype == "bf16":
        Q, K, V = bf16_round(Q), bf16_round(K), bf16_round(V)
    return Q, K, V


def make_pairs(npairs: int, d: int = 64, seed: int = 4000):
    """The variance-study pairs: entries Uniform[0,1], each vector L2-normalised
    and multiplied by 2 (float32)."""
    X = _rng(seed, 1).random((npairs, d), dtype=np.float32)
    Y = _rng(seed, 2).random((npairs, d), dtype=np.float32)
    X *= np.float32(2.0) / np.linalg.norm(X, axis=1, keepdims=True).astype(np.float32)
    Y *= np.float32(2.0) / np.linalg.norm(Y, axis=1, keepdims=True).astype(np.float32)
    return X, Y


@dataclass(frozen=True)
class PairWorkload:
    """The variance-study batch: npairs (x, y) pairs, R independent draws of M orthogonal features shared by
    all pairs, one parameter fit per variant over all the x's and y's."""
    name: str
    npairs: int
    d: int
    M: int
    R: int
    variants: tuple
    seed: int = 4000

    def scaled(self, **kw) -> "PairWorkload":
        return replace(self, **kw)


PAIR_WORKLOADS = {
    "cfg4": PairWorkload("cfg4", 2 ** 20, 64, 64, 32, ("aderf", "sderf", "gerf", "posrf")),
}


def make_pair_omegas(pw: PairWorkload) -> np.ndarray:
    """(R, M, d): draw r is an orthogonal block of its own (seed + r)."""
    return np.stack([orthogonal_omega(pw.M, pw.d, pw.seed + r) for r in range(pw.R)])
