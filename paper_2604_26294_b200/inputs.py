"""Seeded synthetic inputs for the TSP gated-MLP path.

This module holds no arithmetic of the method itself: it draws random numbers,
rounds them to bf16 bit patterns and rearranges memory layouts.  Both the CPU
oracle's tests and the CUDA path's tests/bench read their inputs from here so
that the two sides see exactly the same bits.

Recipe (fixed; any change invalidates stored comparisons):
  * generator  numpy ``Generator(Philox(seed))``
  * draw order ``X, Wg, Wu, Wd, dY`` as float32 standard normals, scaled by the
    standard deviations below, then rounded to bf16 (round-to-nearest-even)
  * ``X  ~ N(0, 1)``            shape [S, H]
  * ``Wg, Wu ~ N(0, var 1/H)``  shape [H, F]   (unsharded; shard k = columns k*F/D..)
  * ``Wd ~ N(0, var 1/F)``      shape [F, H]   (unsharded; shard k = rows    k*F/D..)
  * ``dY ~ N(0, 1)``            shape [S, H]   (only when ``with_dy``)
The unsharded matrices do not depend on D, so the same seed gives the same
mathematical problem for every shard count.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Workload:
    """One problem size: S tokens in total, hidden H, intermediate width F, D shards."""

    name: str
    S: int
    H: int
    F: int
    D: int

    @property
    def S_loc(self) -> int:
        return self.S // self.D

    @property
    def F_d(self) -> int:
        return self.F // self.D

    def forward_flops(self) -> float:
        """Model FLOPs of the forward gated MLP: three S x H x F contractions."""
        return 6.0 * self.S * self.H * self.F

    def backward_flops(self) -> float:
        """Model FLOPs of the backward pass (twice the forward, no recompute counted)."""
        return 12.0 * self.S * self.H * self.F


# The named workloads.  "tiny" is the one the CPU oracle finishes in well under a
# second; the 7B-shaped ones use H=4096, F=14336.
WORKLOADS = {
    "tiny": Workload("tiny", S=256, H=256, F=768, D=2),
    "7b_short": Workload("7b_short", S=8192, H=4096, F=14336, D=8),
    "7b_long": Workload("7b_long", S=65536, H=4096, F=14336, D=8),
    "sweep_d1": Workload("sweep_d1", S=16384, H=4096, F=14336, D=1),
    "sweep_d2": Workload("sweep_d2", S=16384, H=4096, F=14336, D=2),
    "sweep_d4": Workload("sweep_d4", S=16384, H=4096, F=14336, D=4),
    "sweep_d8": Workload("sweep_d8", S=16384, H=4096, F=14336, D=8),
    "sweep_d16": Workload("sweep_d16", S=16384, H=4096, F=14336, D=16),
    "train": Workload("train", S=8192, H=4096, F=14336, D=8),
    # the paper's own 7B-class MLP: expansion factor 4, intermediate width 4 * 4096 (reference-model table)
    "7b_paper": Workload("7b_paper", S=8192, H=4096, F=16384, D=8),
    # a larger model shape (hidden 8192, intermediate 28672) to exercise other H / F than the 7B ones
    "70b_short": Workload("70b_short", S=4096, H=8192, F=28672, D=8),
}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 with round-to-nearest-even; returns uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    # NaNs are not produced by the generator; plain RNE on the upper 16 bits.
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float32 exactly."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to float64 exactly."""
    return bf16_bits_to_f32(bits).astype(np.float64)


def _draw_bf16(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    rows = shape[0]
    out = np.empty(shape, dtype=np.uint16)
    # Drawn in row blocks so the float32 temporary stays small at the long-context sizes;
    # the stream of normals is the same as one big draw.
    step = max(1, (1 << 24) // max(1, int(np.prod(shape[1:]))))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        blk = rng.standard_normal((r1 - r0,) + tuple(shape[1:]), dtype=np.float32)
        if std != 1.0:
            blk *= np.float32(std)
        out[r0:r1] = f32_to_bf16_bits(blk)
    return out


@dataclass
class Inputs:
    """bf16 bit patterns (uint16) of one seeded problem, unsharded layouts."""

    X: np.ndarray  # [S, H]
    Wg: np.ndarray  # [H, F]
    Wu: np.ndarray  # [H, F]
    Wd: np.ndarray  # [F, H]
    dY: np.ndarray | None  # [S, H]


def make_inputs(S: int, H: int, F: int, seed: int = 0, with_dy: bool = False) -> Inputs:
    rng = np.random.Generator(np.random.Philox(seed))
    X = _draw_bf16(rng, (S, H), 1.0)
    Wg = _draw_bf16(rng, (H, F), H ** -0.5)
    Wu = _draw_bf16(rng, (H, F), H ** -0.5)
    Wd = _draw_bf16(rng, (F, H), F ** -0.5)
    dY = _draw_bf16(rng, (S, H), 1.0) if with_dy else None
    return Inputs(X, Wg, Wu, Wd, dY)


def shard_columns(W: np.ndarray, D: int) -> np.ndarray:
    """[H, F] -> [D, H, F/D]: shard k holds columns k*F/D .. (k+1)*F/D (gate / up layout)."""
    H, F = W.shape
    assert F % D == 0
    return np.ascontiguousarray(W.reshape(H, D, F // D).transpose(1, 0, 2))


def unshard_columns(Wk: np.ndarray) -> np.ndarray:
    """[D, H, F/D] -> [H, F]; inverse of :func:`shard_columns`."""
    D, H, Fd = Wk.shape
    return np.ascontiguousarray(Wk.transpose(1, 0, 2).reshape(H, D * Fd))


def shard_rows(W: np.ndarray, D: int) -> np.ndarray:
    """[F, H] -> [D, F/D, H]: shard k holds rows k*F/D .. (k+1)*F/D (down layout; a pure reshape)."""
    F, H = W.shape
    assert F % D == 0
    return np.ascontiguousarray(W.reshape(D, F // D, H))


def unshard_rows(Wk: np.ndarray) -> np.ndarray:
    """[D, F/D, H] -> [F, H]; inverse of :func:`shard_rows`."""
    D, Fd, H = Wk.shape
    return np.ascontiguousarray(Wk.reshape(D * Fd, H))


def sample_rows(S: int, D: int, block: int = 128, per_block: int = 1, seed: int = 1) -> np.ndarray:
    """Row indices with `per_block` random rows inside every `block`-row tile of every rank."""
    rng = np.random.Generator(np.random.Philox(seed))
    rows = []
    for b0 in range(0, S, block):
        n = min(block, S - b0)
        rows.extend(b0 + rng.choice(n, size=min(per_block, n), replace=False))
    return np.sort(np.asarray(rows, dtype=np.int64))


def sample_columns(F: int, D: int, count: int, seed: int = 2) -> np.ndarray:
    """`count` intermediate-column indices, spread so that every shard k is hit."""
    rng = np.random.Generator(np.random.Philox(seed))
    F_d = F // D
    per = max(1, count // D)
    cols = []
    for k in range(D):
        cols.extend(k * F_d + rng.choice(F_d, size=min(per, F_d), replace=False))
    return np.sort(np.asarray(cols, dtype=np.int64))


# ----------------------------------------------------------------------------------------
# Projection GEMMs of TSP attention (Algorithm 1): seeded inputs only, no arithmetic of the method.
# ----------------------------------------------------------------------------------------
@dataclass(frozen=True)
class AttnWorkload:
    """S tokens, hidden H, query width Hq = n_heads * head_dim, key/value width Hkv = Hq / g, D shards."""

    name: str
    S: int
    H: int
    Hq: int
    Hkv: int
    D: int

    def qkv_flops(self) -> float:
        return 2.0 * self.S * self.H * (self.Hq + 2 * self.Hkv)

    def out_flops(self) -> float:
        return 2.0 * self.S * self.Hq * self.H


ATTN_WORKLOADS = {
    "attn_tiny": AttnWorkload("attn_tiny", S=256, H=256, Hq=512, Hkv=256, D=2),
    # 7B-class layer of the reference-model table: h = 4096, 32 heads of 128; MHA and a GQA variant (g = 4)
    "attn_7b_mha": AttnWorkload("attn_7b_mha", S=8192, H=4096, Hq=4096, Hkv=4096, D=8),
    "attn_7b_gqa4": AttnWorkload("attn_7b_gqa4", S=8192, H=4096, Hq=4096, Hkv=1024, D=8),
    "attn_7b_long": AttnWorkload("attn_7b_long", S=65536, H=4096, Hq=4096, Hkv=4096, D=8),
}


@dataclass
class AttnInputs:
    """bf16 bit patterns (uint16), unsharded layouts (rows of the weights = output features)."""

    X: np.ndarray   # [S, H]
    Wq: np.ndarray  # [Hq, H]
    Wk: np.ndarray  # [Hkv, H]
    Wv: np.ndarray  # [Hkv, H]
    A: np.ndarray   # [S, Hq]   stand-in for the attention output fed to the output projection
    Wo: np.ndarray  # [H, Hq]
    dQ: np.ndarray | None = None  # [S, Hq]   upstream gradients (stand-ins for what attention's backward hands over)
    dK: np.ndarray | None = None  # [S, Hkv]
    dV: np.ndarray | None = None  # [S, Hkv]
    dY: np.ndarray | None = None  # [S, H]


def make_attn_inputs(S: int, H: int, Hq: int, Hkv: int, seed: int = 0, with_grads: bool = False) -> AttnInputs:
    """Draw order X, Wq, Wk, Wv, A, Wo (then dQ, dK, dV, dY); X, A, gradients ~ N(0,1); Wq, Wk, Wv ~ N(0, var 1/H);
    Wo ~ N(0, var 1/Hq)."""
    rng = np.random.Generator(np.random.Philox(seed))
    X = _draw_bf16(rng, (S, H), 1.0)
    Wq = _draw_bf16(rng, (Hq, H), H ** -0.5)
    Wk = _draw_bf16(rng, (Hkv, H), H ** -0.5)
    Wv = _draw_bf16(rng, (Hkv, H), H ** -0.5)
    A = _draw_bf16(rng, (S, Hq), 1.0)
    Wo = _draw_bf16(rng, (H, Hq), Hq ** -0.5)
    out = AttnInputs(X, Wq, Wk, Wv, A, Wo)
    if with_grads:
        out.dQ = _draw_bf16(rng, (S, Hq), 1.0)
        out.dK = _draw_bf16(rng, (S, Hkv), 1.0)
        out.dV = _draw_bf16(rng, (S, Hkv), 1.0)
        out.dY = _draw_bf16(rng, (S, H), 1.0)
    return out


def shard_out_columns(Wo: np.ndarray, D: int) -> np.ndarray:
    """[H, Hq] -> [D, H, Hq/D]: shard r of the output projection holds the columns of shard r's heads."""
    return shard_columns(Wo, D)
