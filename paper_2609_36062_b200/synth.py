"""Seeded synthetic inputs shaped like the paper's prefill workloads.

This module holds no arithmetic of the method: it only draws Q, K, V (and an upstream
gradient dO) from a counter-based generator and rounds them to the storage dtype.  It is
the single piece that both the CUDA path and the CPU oracle's tests read, so that the
two see identical bytes.

Recipe.  Every (tensor, batch·head) pair owns its own Philox stream keyed by
(seed, tensor id, head index), so one head can be regenerated without the others.
  * "scaled":     Q, K, V iid N(0,1)/sqrt(d)                         (fp32 small case)
  * "normalised": Q, K iid N(0,1)/sqrt(d_k), then every row L2-normalised in fp32;
                  V iid N(0,1)
  * "positive":   Q, K iid |N(0,1)|/sqrt(d_k) (non-negative features for the normalised output); V iid N(0,1)
  * dO iid N(0,1)
bf16 storage rounds the fp32 values once, to nearest even; the oracle widens exactly
those rounded values to fp64.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_TENSOR_ID = {"q": 0, "k": 1, "v": 2, "do": 3}


@dataclass(frozen=True)
class Workload:
    name: str
    d: int            # VC dimension of the mask family member
    batch: int
    heads: int
    T: int
    d_k: int
    d_v: int
    chunk: int
    dtype: str        # "f32" or "bf16"
    recipe: str       # "scaled" or "normalised"
    seed: int
    backward: bool = False
    routing: str = "positional"   # or "hashed": prof / type arrays drawn by a fixed random hash (user-supplied routing)
    variant: str = "plain"        # "gated": scalar per-token gates; "normalized": augmented ones column and division

    @property
    def bh(self) -> int:
        return self.batch * self.heads

    @property
    def tokens(self) -> int:
        return self.batch * self.T


# The five benchmark configurations (index 0 is the small case an fp64 CPU check finishes in seconds).
WORKLOADS = {
    "small_d2":      Workload("small_d2", 2, 1, 1, 512, 64, 64, 64, "f32", "scaled", 0),
    "small_d1":      Workload("small_d1", 1, 1, 1, 512, 64, 64, 64, "f32", "scaled", 0),
    "t4k_d3":        Workload("t4k_d3", 3, 4, 8, 4096, 128, 128, 64, "bf16", "normalised", 1),
    "t16k_d4":       Workload("t16k_d4", 4, 2, 16, 16384, 128, 128, 128, "bf16", "normalised", 2),
    "t64k_d1":       Workload("t64k_d1", 1, 1, 16, 65536, 128, 128, 128, "bf16", "normalised", 3),
    "t64k_d2":       Workload("t64k_d2", 2, 1, 16, 65536, 128, 128, 128, "bf16", "normalised", 3),
    "t64k_d3":       Workload("t64k_d3", 3, 1, 16, 65536, 128, 128, 128, "bf16", "normalised", 3),
    "t64k_d4":       Workload("t64k_d4", 4, 1, 16, 65536, 128, 128, 128, "bf16", "normalised", 3),
    # reduced-head copies of two workloads, small enough to profile kernel by kernel (tables still exceed L2)
    "t16k_d4_h2":    Workload("t16k_d4_h2", 4, 1, 2, 16384, 128, 128, 128, "bf16", "normalised", 2),
    "t16k_d4_h8":    Workload("t16k_d4_h8", 4, 1, 8, 16384, 128, 128, 128, "bf16", "normalised", 2),
    "t64k_d4_h1":    Workload("t64k_d4_h1", 4, 1, 1, 65536, 128, 128, 128, "bf16", "normalised", 3),
    "t64k_d3_h2":    Workload("t64k_d3_h2", 3, 1, 2, 65536, 128, 128, 128, "bf16", "normalised", 3),
    "t64k_d3_h4":    Workload("t64k_d3_h4", 3, 1, 4, 65536, 128, 128, 128, "bf16", "normalised", 3),
    "t8k_d3_h8":     Workload("t8k_d3_h8", 3, 1, 8, 8192, 128, 128, 64, "bf16", "normalised", 4),
    "t64k_d1_h4":    Workload("t64k_d1_h4", 1, 1, 4, 65536, 128, 128, 128, "bf16", "normalised", 3),
    "t64k_d2_h4":    Workload("t64k_d2_h4", 2, 1, 4, 65536, 128, 128, 128, "bf16", "normalised", 3),
    "t8k_d3_fwdbwd": Workload("t8k_d3_fwdbwd", 3, 8, 16, 8192, 128, 128, 64, "bf16", "normalised", 4, True),
    "t8k_d3_h16_fwdbwd": Workload("t8k_d3_h16_fwdbwd", 3, 1, 16, 8192, 128, 128, 64, "bf16", "normalised", 4, True),
    # the 16 K configuration under user-supplied routing: every token hashed to a uniformly random cell / type
    "t16k_d4_hashed": Workload("t16k_d4_hashed", 4, 2, 16, 16384, 128, 128, 128, "bf16", "normalised", 2, False, "hashed"),
    # the variants of the "next" list on benchmark-shaped inputs
    "t4k_d3_gated":  Workload("t4k_d3_gated", 3, 4, 8, 4096, 128, 128, 64, "bf16", "normalised", 1, False, "positional", "gated"),
    "t4k_d3_gated_fwdbwd": Workload("t4k_d3_gated_fwdbwd", 3, 4, 8, 4096, 128, 128, 64, "bf16", "normalised", 1, True,
                                    "positional", "gated"),
    "t16k_d4_normalized": Workload("t16k_d4_normalized", 4, 2, 16, 16384, 128, 128, 128, "bf16", "positive", 2, False,
                                   "positional", "normalized"),
    # cached decoding: 128 sequences of 16 heads, 2 K horizon (132 type states + one running state per head; the
    # running states alone, 134 MB, exceed L2)
    "decode_t2k_d3": Workload("decode_t2k_d3", 3, 128, 16, 2048, 128, 128, 64, "bf16", "normalised", 5),
    "decode_t2k_d3_b32": Workload("decode_t2k_d3_b32", 3, 32, 16, 2048, 128, 128, 64, "bf16", "normalised", 5),
}


def _stream(seed: int, tensor: str, head: int) -> np.random.Generator:
    key = (int(seed) << 40) ^ (_TENSOR_ID[tensor] << 32) ^ int(head)
    return np.random.Generator(np.random.Philox(key=key))


def bf16_round(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit pattern (uint16), round to nearest even.  Inputs are finite."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


def bf16_widen(b: np.ndarray) -> np.ndarray:
    """bf16 bit pattern (uint16) -> the same value as fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def head_tensor(w: Workload, tensor: str, head: int, T: int | None = None) -> np.ndarray:
    """fp32 values of one [T, dim] slice before storage rounding."""
    T = w.T if T is None else T
    dim = w.d_v if tensor in ("v", "do") else w.d_k
    x = _stream(w.seed, tensor, head).standard_normal((T, dim), dtype=np.float32)
    if tensor == "do":
        return x
    if w.recipe == "scaled":
        return x * np.float32(1.0 / np.sqrt(dim))
    if w.recipe == "positive":      # non-negative features (normalised output): half-normal Q, K; V iid N(0,1)
        return (np.abs(x) * np.float32(1.0 / np.sqrt(dim))).astype(np.float32) if tensor in ("q", "k") else x
    if tensor in ("q", "k"):
        x = x * np.float32(1.0 / np.sqrt(dim))
        norm = np.sqrt(np.sum(x * x, axis=1, keepdims=True, dtype=np.float32))
        return (x / norm).astype(np.float32)
    return x


def stored(w: Workload, tensor: str, head: int) -> np.ndarray:
    """One head in its storage form: fp32 array, or uint16 array of bf16 bit patterns."""
    x = head_tensor(w, tensor, head)
    return x if w.dtype == "f32" else bf16_round(x)


def as_float64(w: Workload, stored_head: np.ndarray) -> np.ndarray:
    """The exact stored values widened to fp64 (what the oracle computes on)."""
    if w.dtype == "f32":
        return stored_head.astype(np.float64)
    return bf16_widen(stored_head).astype(np.float64)


def full_tensor(w: Workload, tensor: str) -> np.ndarray:
    """All heads: shape [batch*heads, T, dim] in storage form."""
    return np.stack([stored(w, tensor, h) for h in range(w.bh)])


def hashed_cells(w: Workload, head: int, n: int, P: int, skew: float = 0.0) -> np.ndarray:
    """A fixed random hash of the distant tokens of one head into P cells (int32 [n]): uniform, or, with skew > 0,
    drawn from a power law so that a few cells are heavy and many are empty."""
    g = np.random.Generator(np.random.Philox(key=(int(w.seed) << 40) ^ (7 << 32) ^ int(head)))
    if skew <= 0:
        return g.integers(0, P, size=n, dtype=np.int64).astype(np.int32)
    weights = 1.0 / np.arange(1, P + 1, dtype=np.float64) ** skew
    perm = g.permutation(P)
    return perm[g.choice(P, size=n, p=weights / weights.sum())].astype(np.int32)


def hashed_query_draws(w: Workload, head: int, m: int, P: int, A: int) -> tuple[np.ndarray, np.ndarray]:
    """Per recent token of one head: a hashed cell in [0, P) and a direction number in [0, A) (both int32 [m]); the
    type that goes with them (the hyperplane of that direction through that cell) is the method's arithmetic and is
    computed by whoever uses the draws."""
    g = np.random.Generator(np.random.Philox(key=(int(w.seed) << 40) ^ (8 << 32) ^ int(head)))
    return (g.integers(0, P, size=m, dtype=np.int64).astype(np.int32),
            g.integers(0, A, size=m, dtype=np.int64).astype(np.int32))


def hashed_types(w: Workload, head: int, m: int, B: int) -> np.ndarray:
    """A fixed random hash of the recent tokens of one head into B types (int32 [m]), uniform."""
    g = np.random.Generator(np.random.Philox(key=(int(w.seed) << 40) ^ (9 << 32) ^ int(head)))
    return g.integers(0, B, size=m, dtype=np.int64).astype(np.int32)


def log_gates(w: Workload, head: int, lo: float = 0.9) -> np.ndarray:
    """Per-token log-gates of one head (fp32 [T]): gates uniform in [lo, 1)."""
    g = np.random.Generator(np.random.Philox(key=(int(w.seed) << 40) ^ (10 << 32) ^ int(head)))
    return np.log(g.uniform(lo, 1.0, size=w.T)).astype(np.float32)
