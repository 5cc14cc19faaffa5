"""Seeded synthetic inputs for the contrastive-loss hot path.

This module only *generates data*: representation matrices Q (B x d), P (N x d) and the
relevance map pos_idx (the paper's r_i, Section 3.1).  It holds none of the method's
arithmetic (no similarity, softmax, loss or gradient), so that the CPU checker and the CUDA
path can both be fed from it without sharing any computation.

Random numbers come from numpy's Philox generator (a counter-based PRNG) keyed by the seed.
The paper's workloads are question/passage batches encoded by BERT (d = 768) with one positive
and one hard negative passage per question (Section 4); that data is not available, so the
recipes below reproduce its shapes and the typical similarity structure (a positive that is
close to the query, a hard negative that is less close, everything else near-orthogonal).
"""
from __future__ import annotations

import dataclasses

import numpy as np

MASK_NONE = 0
MASK_SELF = 1

BASE_SEED = 2101069830


@dataclasses.dataclass
class Problem:
    """One problem instance.  Q and P are float32 arrays whose values are exactly representable
    in `dtype` ("f32" or "bf16"); for bf16 the raw 16-bit patterns are in Q_bits / P_bits."""
    name: str
    Q: np.ndarray
    P: np.ndarray
    pos_idx: np.ndarray
    tau: float
    mask_mode: int
    dtype: str
    shared: bool = False          # True when Q and P are the same rows (symmetric loss)
    Q_bits: np.ndarray | None = None
    P_bits: np.ndarray | None = None

    @property
    def B(self) -> int:
        return int(self.Q.shape[0])

    @property
    def N(self) -> int:
        return int(self.P.shape[0])

    @property
    def d(self) -> int:
        return int(self.Q.shape[1])


def bf16_round(x: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """Round float32 to bfloat16 (round to nearest, ties to even).
    Returns (uint16 bit patterns, the rounded values widened back to float32)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    nan = np.isnan(x)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = (u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)
    bits = r.astype(np.uint32)
    bits[nan] = 0x7FC0
    bits16 = bits.astype(np.uint16)
    back = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return bits16, back.reshape(x.shape)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=int(seed)))


def _normal(rng: np.random.Generator, shape, sigma: float) -> np.ndarray:
    out = rng.standard_normal(size=shape, dtype=np.float32)
    out *= np.float32(sigma)
    return out


def _finish(name, Q, P, pos, tau, mask_mode, dtype, shared=False) -> Problem:
    if dtype == "bf16":
        qb, Q = bf16_round(Q)
        if shared:
            pb, P = qb, Q
        else:
            pb, P = bf16_round(P)
        return Problem(name, Q, P, pos, tau, mask_mode, dtype, shared, qb, pb)
    if dtype != "f32":
        raise ValueError(f"unknown dtype {dtype!r}")
    Q = np.ascontiguousarray(Q, dtype=np.float32)
    P = Q if shared else np.ascontiguousarray(P, dtype=np.float32)
    return Problem(name, Q, P, pos, tau, mask_mode, dtype, shared)


def dpr_batch(B: int, d: int = 768, dtype: str = "bf16", seed: int = BASE_SEED,
              tau: float = 1.0, name: str | None = None) -> Problem:
    """Retrieval-style batch: B queries, N = 2B passages.  Passage 2i is query i's positive,
    passage 2i+1 its hard negative, every other passage an in-batch negative.

    q_i ~ N(0, sigma^2 I) with sigma = d**-0.5 (so |q_i| is about 1);
    positive = 0.8 q_i + 0.6 z_i, hard negative = 0.5 q_i + 0.866 z'_i, z and z' drawn like q.
    """
    rng = _rng(seed)
    sigma = float(d) ** -0.5
    N = 2 * B
    Q = np.empty((B, d), np.float32)
    P = np.empty((N, d), np.float32)
    step = 8192
    for lo in range(0, B, step):
        hi = min(B, lo + step)
        q = _normal(rng, (hi - lo, d), sigma)
        z = _normal(rng, (hi - lo, d), sigma)
        z2 = _normal(rng, (hi - lo, d), sigma)
        Q[lo:hi] = q
        P[2 * lo:2 * hi:2] = np.float32(0.8) * q + np.float32(0.6) * z
        P[2 * lo + 1:2 * hi:2] = np.float32(0.5) * q + np.float32(0.866) * z2
    pos = (2 * np.arange(B, dtype=np.int64)).astype(np.int32)
    return _finish(name or f"dpr_B{B}_d{d}_{dtype}", Q, P, pos, tau, MASK_NONE, dtype)


def simclr_batch(M: int, d: int = 128, dtype: str = "bf16", seed: int = BASE_SEED + 3,
                 tau: float = 0.1, noise: float = 0.3, name: str | None = None) -> Problem:
    """Symmetric two-view batch: 2M rows, rows 0..M-1 are view a, M..2M-1 view b of M items.
    view = x + noise * n, L2-normalised in float32.  Q and P are the same 2M rows, the
    self-similarity diagonal is masked, and row i's positive is its partner view."""
    rng = _rng(seed)
    x = _normal(rng, (M, d), 1.0)
    a = x + np.float32(noise) * _normal(rng, (M, d), 1.0)
    b = x + np.float32(noise) * _normal(rng, (M, d), 1.0)
    X = np.concatenate([a, b], axis=0)
    X /= np.sqrt((X.astype(np.float64) ** 2).sum(axis=1, keepdims=True)).astype(np.float32)
    pos = ((np.arange(2 * M, dtype=np.int64) + M) % (2 * M)).astype(np.int32)
    return _finish(name or f"simclr_M{M}_d{d}_{dtype}", X, X, pos, tau, MASK_SELF, dtype,
                   shared=True)


def random_problem(B: int, N: int, d: int, dtype: str = "f32", seed: int = 0, tau: float = 1.0,
                   mask_mode: int = MASK_NONE, scale: float = 1.0, shared: bool = False,
                   duplicates: bool = True) -> Problem:
    """Unstructured problem for edge-case tests: iid normal entries of standard deviation
    `scale`, random positives (with repeats allowed when `duplicates`).  Under MASK_SELF the
    positive of row i is never column i."""
    rng = _rng(seed)
    Q = _normal(rng, (B, d), scale)
    if shared:
        if B != N:
            raise ValueError("shared rows need B == N")
        P = Q
    else:
        P = _normal(rng, (N, d), scale)
    if duplicates:
        pos = rng.integers(0, N, size=B, dtype=np.int64)
    else:
        pos = rng.permutation(N)[:B].astype(np.int64)
    if mask_mode == MASK_SELF:
        i = np.arange(B, dtype=np.int64)
        clash = pos == i
        pos[clash] = (pos[clash] + 1) % N
    return _finish(f"rand_B{B}_N{N}_d{d}_{dtype}_s{seed}", Q, P, pos.astype(np.int32), tau,
                   mask_mode, dtype, shared)


def config(index: int) -> Problem:
    """The five named workloads (seed = BASE_SEED + index)."""
    s = BASE_SEED + index
    if index == 0:
        return dpr_batch(64, 768, "f32", s, name="cfg0_B64_N128_d768_f32")
    if index == 1:
        return dpr_batch(128, 768, "bf16", s, name="cfg1_B128_N256_d768_bf16")
    if index == 2:
        return dpr_batch(4096, 768, "bf16", s, name="cfg2_B4096_N8192_d768_bf16")
    if index == 3:
        return simclr_batch(4096, 128, "bf16", s, name="cfg3_2M8192_d128_bf16_self")
    if index == 4:
        return dpr_batch(65536, 768, "bf16", s, name="cfg4_B65536_N131072_d768_bf16")
    raise ValueError("config index must be 0..4")


def encoder_inputs(rows: int, d_in: int, seed: int = 0, sigma: float = 1.0):
    """Stand-in for the inputs s_i of a linear encoder (Step 3, Eq. 8-9): a [rows x d_in] matrix
    of N(0, sigma^2) values rounded to bf16.  Returns (uint16 bit patterns, float32 values)."""
    return bf16_round(_normal(_rng(BASE_SEED + 1000 + seed), (rows, d_in), sigma))


def cache_rows(rows: int, d: int, seed: int = 0, spread: float = 4.0) -> np.ndarray:
    """Stand-in for rows of a representation gradient cache: float32 values of mixed sign whose
    magnitudes span about 2^(+-spread) around 1/rows (a few rows carry most of the gradient, as
    after a softmax), so that a sloppy low-precision product would show."""
    rng = _rng(BASE_SEED + 2000 + seed)
    mag = np.exp2(rng.uniform(-spread, spread, size=(rows, 1)).astype(np.float32))
    u = rng.standard_normal(size=(rows, d), dtype=np.float32) * mag / np.float32(rows)
    return np.ascontiguousarray(u, dtype=np.float32)
