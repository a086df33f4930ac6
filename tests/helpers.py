"""Shared helpers of the GPU parity tests: move seeded inputs to the device, compare with the oracle."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_36062_b200 import synth

TOL = {"f32": 1e-4, "bf16": 2e-2}   # max|err| / max|ref| bounds stated for the method's outputs and gradients


def to_device(w: synth.Workload, stored: np.ndarray) -> torch.Tensor:
    """[bh, T, dim] storage array -> [batch, heads, T, dim] CUDA tensor of the plan dtype."""
    bh, T, dim = stored.shape
    if w.dtype == "f32":
        t = torch.from_numpy(stored)
    else:
        t = torch.from_numpy(stored.view(np.int16)).view(torch.bfloat16)
    return t.reshape(w.batch, w.heads, T, dim).cuda()


def to_numpy64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def device_inputs(w: synth.Workload, tensors=("q", "k", "v")):
    host = {name: synth.full_tensor(w, name) for name in tensors}
    dev = {name: to_device(w, host[name]) for name in tensors}
    return host, dev


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    denom = float(np.max(np.abs(ref)))
    return float(np.max(np.abs(got - ref))) / (denom if denom > 0 else 1.0)


def sample_tokens(geo, count: int, seed: int) -> list[int]:
    """Token indices that always include both ends, both sides of the block boundary and of chunk
    edges, and one query of each of the first 64 types (types 0..63, each at a different one of its
    occurrences so that the samples spread over the recent block); the rest are drawn at random."""
    T, n, c = geo.T, geo.n, geo.c
    fixed = {0, 1, c - 1, c, n - 1, n, n + 1, n + c - 1, n + c, T - 1, T - c, T - c - 1, n // 2, n + (T - n) // 2}
    B, m = geo.B, T - n
    for h in range(min(64, B)):
        first = h if h >= 1 else B                   # 1-based recent index of the type's first query
        if first > m:
            continue
        occurrences = (m - first) // B + 1
        fixed.add(n + first - 1 + (h % occurrences) * B)
    fixed = {t for t in fixed if 0 <= t < T}
    g = np.random.default_rng(seed)
    extra = g.choice(T, size=max(0, count - len(fixed)), replace=False).tolist() if count > len(fixed) else []
    return sorted(fixed | set(int(t) for t in extra))
