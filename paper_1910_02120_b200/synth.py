"""Seeded synthetic inputs for Independent Subnet Training (IST) workloads.

This module only draws random numbers and lays them out; it contains none of
the method's arithmetic (no partition, no forward/backward, no update).  The
tests and the benchmark call it once and hand the same arrays to every
implementation under comparison.

The shapes follow the paper's experimental settings (Sec. 3, "Experimental
Settings": wide one- and two-hidden-layer MLPs on 35-class speech features,
pixel inputs with 10 classes, and a 135,909-input / 670,091-label extreme
classification network); the datasets themselves are replaced by i.i.d. draws
of the same shape and value distribution.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional, Tuple

import numpy as np

BASE_SEED = 1234


@dataclass(frozen=True)
class Workload:
    """One IST workload: network shape, partition count and data recipe."""

    name: str
    layer_dims: Tuple[int, ...]      # N_0 .. N_t
    S: int                           # number of subnets (the paper's n)
    B: int                           # minibatch rows per subnet per local step
    K: int                           # local SGD steps per round (the paper's J)
    rounds: int
    precision: str                   # "fp32" or "bf16" (operand precision)
    x_dist: str                      # "normal" | "uniform_std" | "csr"
    lr: float = 0.01
    seed: int = BASE_SEED
    csr_mean_nnz: float = 75.0

    @property
    def n_classes(self) -> int:
        return self.layer_dims[-1]

    @property
    def samples_per_round(self) -> int:
        return self.S * self.K * self.B

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five workload families (index = position in the benchmark's config list).
C1 = Workload("C1-tiny-fp32", (784, 1024, 10), S=2, B=128, K=10, rounds=1,
              precision="fp32", x_dist="normal", seed=BASE_SEED + 0)
C2 = Workload("C2-speech-like", (1024, 4096, 4096, 35), S=4, B=256, K=50, rounds=20,
              precision="bf16", x_dist="normal", seed=BASE_SEED + 1)
C3 = Workload("C3-wide-pixels", (3072, 16384, 16384, 10), S=8, B=512, K=20, rounds=10,
              precision="bf16", x_dist="uniform_std", seed=BASE_SEED + 2)
C4 = Workload("C4-extreme-csr", (135909, 1024, 670091), S=8, B=256, K=10, rounds=1,
              precision="bf16", x_dist="csr", seed=BASE_SEED + 3)


def c5(H: int, S: int, K: int) -> Workload:
    return Workload(f"C5-sweep-H{H}-S{S}-K{K}", (1024, H, H, 100), S=S, B=512, K=K,
                    rounds=1, precision="bf16", x_dist="normal", seed=BASE_SEED + 4)


WORKLOADS = {"C1": C1, "C2": C2, "C3": C3, "C4": C4}


def rng_for(seed: int, stream: int) -> np.random.Generator:
    """Independent PCG64 stream per (seed, purpose)."""
    return np.random.Generator(np.random.PCG64([int(seed), int(stream)]))


def make_weights(layer_dims, seed: int, bias_scale: float = 0.0):
    """Full-network parameters: W_l is [N_{l-1}][N_l] (y = x @ W_l + b_l), fp32.

    W ~ U(-sqrt(6/fan_in), +sqrt(6/fan_in)); biases are zero unless
    `bias_scale` asks for U(-bias_scale, +bias_scale) (used by tests so that the
    bias path is exercised).
    """
    Ws: List[np.ndarray] = []
    bs: List[np.ndarray] = []
    for l in range(1, len(layer_dims)):
        fan_in, fan_out = int(layer_dims[l - 1]), int(layer_dims[l])
        g = rng_for(seed, 100 + l)
        bound = np.sqrt(6.0 / fan_in)
        W = g.random((fan_in, fan_out), dtype=np.float32)
        W *= np.float32(2.0 * bound)
        W -= np.float32(bound)
        Ws.append(W)
        if bias_scale > 0.0:
            b = (g.random(fan_out, dtype=np.float32) * 2.0 - 1.0) * np.float32(bias_scale)
            bs.append(b.astype(np.float32))
        else:
            bs.append(np.zeros(fan_out, dtype=np.float32))
    return Ws, bs


def make_labels(shape, n_classes: int, seed: int) -> np.ndarray:
    return rng_for(seed, 7).integers(0, n_classes, size=shape, dtype=np.int32)


def make_teacher_task(n_rows: int, N0: int, n_classes: int, seed: int, hidden: int = 32):
    """A learnable classification task: X ~ N(0, 1) [n_rows][N0] fp32 and labels drawn by a fixed
    random scoring function, y = argmax(tanh(X A / sqrt(N0)) C) with A [N0][hidden], C
    [hidden][n_classes] ~ N(0, 1).  Stands in for a real dataset in multi-round runs (labels
    that depend on the inputs, unlike make_labels)."""
    g = rng_for(seed, 11)
    X = g.standard_normal((n_rows, N0), dtype=np.float32)
    A = g.standard_normal((N0, hidden))
    C = g.standard_normal((hidden, n_classes))
    scores = np.tanh(X.astype(np.float64) @ A / np.sqrt(N0)) @ C
    return X, scores.argmax(axis=1).astype(np.int32)


def draw_round_rows(n_rows: int, S: int, K: int, B: int, seed: int, round_index: int) -> np.ndarray:
    """Row indices [S][K][B] of the minibatches of one round: uniform draws without replacement
    inside a batch, independent across subnets, steps and rounds."""
    g = rng_for(seed, 1000 + round_index)
    out = np.empty((S, K, B), dtype=np.int64)
    for s in range(S):
        for k in range(K):
            out[s, k] = g.choice(n_rows, size=B, replace=False)
    return out


def make_dense_inputs(S: int, K: int, B: int, N0: int, dist: str, seed: int) -> np.ndarray:
    """X laid out as [S][K][B][N0] fp32: one distinct batch per subnet per step."""
    g = rng_for(seed, 3)
    if dist == "normal":
        X = g.standard_normal((S, K, B, N0), dtype=np.float32)
    elif dist == "uniform_std":
        X = g.random((S, K, B, N0), dtype=np.float32)
        flat = X.reshape(-1, N0)
        mu = flat.mean(axis=0, dtype=np.float64)
        sd = flat.std(axis=0, dtype=np.float64)
        flat -= mu.astype(np.float32)
        flat /= np.maximum(sd, 1e-12).astype(np.float32)
    else:
        raise ValueError(f"unknown dense distribution {dist!r}")
    return X


def make_csr_inputs(n_rows: int, N0: int, mean_nnz: float, seed: int):
    """CSR matrix with Poisson(mean_nnz) (at least 1) nonzeros per row at distinct,
    sorted, uniformly random columns; values |N(0,1)|.

    Returns (row_ptr int64 [n_rows+1], col int32 [nnz], val fp32 [nnz]).
    """
    g = rng_for(seed, 5)
    counts = np.clip(g.poisson(mean_nnz, size=n_rows), 1, N0).astype(np.int64)
    row_ptr = np.zeros(n_rows + 1, dtype=np.int64)
    np.cumsum(counts, out=row_ptr[1:])
    nnz = int(row_ptr[-1])
    col = np.empty(nnz, dtype=np.int32)
    for r in range(n_rows):
        c = int(counts[r])
        if c * 8 < N0:
            # rejection: draw, de-duplicate, top up (cheap when c << N0)
            picked = np.unique(g.integers(0, N0, size=c, dtype=np.int64))
            while picked.size < c:
                extra = g.integers(0, N0, size=c - picked.size, dtype=np.int64)
                picked = np.unique(np.concatenate([picked, extra]))
        else:
            picked = np.sort(g.choice(N0, size=c, replace=False))
        col[row_ptr[r]:row_ptr[r + 1]] = picked
    val = np.abs(g.standard_normal(nnz, dtype=np.float32))
    return row_ptr, col, val


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bfloat16 (ties to even), returned as fp32.

    Input formatting only: the bf16 workloads feed bf16 features, so every
    implementation must see exactly these values.
    """
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounded = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The uint16 bit patterns of values already on the bf16 grid."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> 16).astype(np.uint16).reshape(x.shape)


@dataclass
class Batchset:
    """Inputs of one round: dense X [S][K][B][N0] or a CSR matrix with S*K*B rows
    (row (s*K + k)*B + b belongs to subnet s, step k), and labels [S][K][B]."""

    y: np.ndarray
    X: Optional[np.ndarray] = None
    row_ptr: Optional[np.ndarray] = None
    col: Optional[np.ndarray] = None
    val: Optional[np.ndarray] = None

    @property
    def is_csr(self) -> bool:
        return self.X is None


def make_round_inputs(w: Workload, round_index: int = 0) -> Batchset:
    seed = w.seed * 1000 + round_index
    y = make_labels((w.S, w.K, w.B), w.n_classes, seed)
    if w.x_dist == "csr":
        rp, col, val = make_csr_inputs(w.S * w.K * w.B, w.layer_dims[0], w.csr_mean_nnz, seed)
        if w.precision == "bf16":
            val = round_to_bf16(val)
        return Batchset(y=y, row_ptr=rp, col=col, val=val)
    X = make_dense_inputs(w.S, w.K, w.B, w.layer_dims[0], w.x_dist, seed)
    if w.precision == "bf16":
        X = round_to_bf16(X)
    return Batchset(y=y, X=X)
