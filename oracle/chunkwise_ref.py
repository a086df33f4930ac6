"""Chunkwise fp64 CPU restatement of the SMat forward and backward algorithms.  TEST INFRASTRUCTURE ONLY.

This is NOT the oracle (that is smat_oracle.py, the dense definition).  It evaluates the
quantities of Algorithm 1 (forward), Algorithm 2 (implicit incidence tabulation) and the
adjoint equations of the chunking proof with the paper's notation, in float64,
one head at a time.  It is checked against the dense oracle in the CPU tests and then
serves two purposes: an independent formula for the same numbers, and a way to look
at the intermediate tables (F, U, D, S_in and their adjoints) when a GPU kernel is wrong.
It shares no code with the CUDA library.

Notation (paper -> here), with identity feature maps and no normaliser:
  φ_i = q_i, ψ_j = k_j, Z_j = k_j v_jᵀ (r x p);  F_x profile table; U_h type table;
  D_b chunk summaries; S_in[b] incoming states; bars denote adjoints.
"""
from __future__ import annotations

import numpy as np

from . import smat_oracle as so


def _chunks(geo):
    """Chunk boundaries: [0,n) and [n,T) are partitioned separately (Sec. 3.1, causal branch)."""
    c = geo.c
    out = []
    for lo, hi in ((0, geo.n), (geo.n, geo.T)):
        s = lo
        while s < hi:
            out.append((s, min(s + c, hi), lo))
            s += c
    return out


def _point_digits(geo):
    """All points of F_q^D as an integer array [P, D]; row v holds the little-endian base-q digits of v."""
    v = np.arange(geo.P, dtype=np.int64)
    return np.stack([(v // geo.q ** ell) % geo.q for ell in range(geo.D)], axis=1)


def tabulate(F, geo):
    """Algorithm 2: U_{a,b} = Σ_{x : aᵀx = b} F_x.  For one direction a the offsets aᵀx split the points into q
    classes; every class is summed into the state of its hyperplane."""
    if geo.dense_G:
        return F.copy()                                   # one point, one hyperplane
    U = np.zeros((geo.B,) + F.shape[1:], dtype=np.float64)
    pts = _point_digits(geo)
    for ai, a in enumerate(so.directions(geo.q, geo.D)):
        offset = (pts @ np.asarray(a, dtype=np.int64)) % geo.q
        for b in range(geo.q):
            U[ai * geo.q + b] = F[offset == b].sum(axis=0)
    return U


def tabulate_transpose(Ubar, geo):
    """F̄ = Cᵀ Ū: a point receives, from every direction, the state of the one hyperplane through it (Eq. lr-adjoint)."""
    if geo.dense_G:
        return Ubar.copy()
    Fbar = np.zeros((geo.P,) + Ubar.shape[1:], dtype=np.float64)
    pts = _point_digits(geo)
    for ai, a in enumerate(so.directions(geo.q, geo.D)):
        offset = (pts @ np.asarray(a, dtype=np.int64)) % geo.q
        Fbar += Ubar[ai * geo.q + offset]
    return Fbar


def _type(t, geo):
    return 0 if geo.dense_G else so.type_index(t, geo)


def _profile(t, geo):
    return 0 if geo.dense_G else t % geo.P


def forward(Q, K, V, geo, return_tables=False):
    """Algorithm 1 without the final division: pooled profile states, tabulated type states, typed read, chunk
    summaries and their exclusive scan per block, per-chunk output."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    T, r = Q.shape
    p = V.shape[1]
    n = geo.n
    # profile table: distant states pooled by profile cell (Eq. schedule)
    F = np.zeros((geo.P, r, p))
    for t in range(n):
        F[_profile(t, geo)] += np.outer(K[t], V[t])
    # type table
    U = tabulate(F, geo)
    # typed read, rows back in chronological order
    Ylr = np.zeros((T, p))
    for t in range(n, T):
        Ylr[t] = Q[t] @ U[_type(t, geo)]
    # chunk summaries and their exclusive scan inside each block (the state restarts at n)
    ch = _chunks(geo)
    Dsum = np.stack([K[s:e].T @ V[s:e] for s, e, _ in ch]) if ch else np.zeros((0, r, p))
    Sin = np.zeros_like(Dsum)
    for b, (s, e, lo) in enumerate(ch):
        if s != lo:
            Sin[b] = Sin[b - 1] + Dsum[b - 1]
    # per-chunk output (Eq. local plus the long-range rows)
    O = np.zeros((T, p))
    for b, (s, e, lo) in enumerate(ch):
        A = np.tril(Q[s:e] @ K[s:e].T)
        O[s:e] = Q[s:e] @ Sin[b] + A @ V[s:e] + Ylr[s:e]
    if return_tables:
        return O, dict(F=F, U=U, D=Dsum, Sin=Sin, Ylr=Ylr)
    return O


def backward(Q, K, V, dO, geo, return_tables=False):
    """Adjoints of every step of Algorithm 1 (chunking proof, backward pass)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    g = np.asarray(dO, dtype=np.float64)
    T, r = Q.shape
    p = V.shape[1]
    n = geo.n
    _, tab = forward(Q, K, V, geo, return_tables=True)
    U, Sin = tab["U"], tab["Sin"]
    dQ = np.zeros((T, r))
    dK = np.zeros((T, r))
    dV = np.zeros((T, p))
    # long-range adjoints
    Ubar = np.zeros_like(U)
    for t in range(n, T):
        h = _type(t, geo)
        Ubar[h] += np.outer(Q[t], g[t])
        dQ[t] += U[h] @ g[t]
    Fbar = tabulate_transpose(Ubar, geo)
    # within-chunk adjoints and the scan adjoint (exclusive suffix scan per block)
    ch = _chunks(geo)
    Sbar = np.stack([Q[s:e].T @ g[s:e] for s, e, _ in ch]) if ch else np.zeros((0, r, p))
    Dbar = np.zeros_like(Sbar)
    for b in range(len(ch) - 1, -1, -1):
        s, e, lo = ch[b]
        last_of_block = (b == len(ch) - 1) or (ch[b + 1][2] != lo)
        if not last_of_block:
            Dbar[b] = Dbar[b + 1] + Sbar[b + 1]
    for b, (s, e, lo) in enumerate(ch):
        A = np.tril(Q[s:e] @ K[s:e].T)
        G = np.tril(g[s:e] @ V[s:e].T)
        dV[s:e] += A.T @ g[s:e]
        dQ[s:e] += g[s:e] @ Sin[b].T + G @ K[s:e]
        dK[s:e] += G.T @ Q[s:e]
    # pointwise: Z̄_j = D̄_{b(j)} (+ F̄_prof(j) for distant j);  ψ̄_j = Z̄_j v_j,  v̄_j = Z̄_jᵀ ψ_j
    for b, (s, e, lo) in enumerate(ch):
        for t in range(s, e):
            Zbar = Dbar[b] + (Fbar[_profile(t, geo)] if t < n else 0.0)
            dK[t] += Zbar @ V[t]
            dV[t] += Zbar.T @ K[t]
    if return_tables:
        return dQ, dK, dV, dict(Ubar=Ubar, Fbar=Fbar, Sbar=Sbar, Dbar=Dbar, **tab)
    return dQ, dK, dV


def streaming_rows(Q, K, V, geo, rows):
    """Streaming evaluation of recent rows: ȳ_{n+i} = φᵀ(U_type(i) + Σ_{n<j<=n+i} Z_j) (decoding proof)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    r, p = Q.shape[1], V.shape[1]
    F = np.zeros((geo.P, r, p))
    for t in range(geo.n):
        F[_profile(t, geo)] += np.outer(K[t], V[t])
    U = tabulate(F, geo)
    want = set(int(t) for t in rows)
    out = {}
    S = np.zeros((r, p))
    for t in range(geo.n, geo.T):
        S += np.outer(K[t], V[t])
        if t in want:
            out[t] = Q[t] @ (U[_type(t, geo)] + S)
    return out


def gated_forward(Q, K, V, log_a, geo):
    """Lemma "Gated SMat": the chunkwise forward under scalar per-token gates.  λ is one prefix sum; every factor is
    exp of a difference λ_i - λ_j with j <= i.  Causal branch: tile entries times exp(λ_i - λ_j), chunk summaries with
    every Z_j scaled to the chunk's last index, the carried state decayed by the chunk's total gate and read with
    exp(λ_i - λ_{e(b-1)}).  Long-range branch: the factor splits at the boundary into a key-side scalar folded into Z_j
    and a query-side scalar on the read; the tables are the ungated ones of rescaled inputs."""
    Q = np.asarray(Q, dtype=np.float64); K = np.asarray(K, dtype=np.float64); V = np.asarray(V, dtype=np.float64)
    lam = np.cumsum(np.asarray(log_a, dtype=np.float64))
    T, r = Q.shape
    p = V.shape[1]
    n = geo.n
    lam_b = lam[n - 1] if n > 0 else 0.0
    F = np.zeros((geo.P, r, p))
    for t in range(n):
        F[_profile(t, geo)] += np.exp(lam_b - lam[t]) * np.outer(K[t], V[t])
    U = tabulate(F, geo)
    O = np.zeros((T, p))
    for t in range(n, T):
        O[t] += np.exp(lam[t] - lam_b) * (Q[t] @ U[_type(t, geo)])
    S = np.zeros((r, p))
    for s, e, lo in _chunks(geo):
        if s == lo:
            S = np.zeros((r, p))                            # the state restarts at the head of each block
        ref = lam[s - 1] if s > 0 else 0.0                  # λ at the last index of the previous chunk
        idx = np.arange(s, e)
        decay = np.exp(np.minimum(lam[idx][:, None] - lam[idx][None, :], 0.0))
        A = np.tril(Q[s:e] @ K[s:e].T) * decay
        O[s:e] += np.exp(lam[idx] - ref)[:, None] * (Q[s:e] @ S) + A @ V[s:e]
        D = (np.exp(lam[e - 1] - lam[idx])[:, None] * K[s:e]).T @ V[s:e]
        S = np.exp(lam[e - 1] - ref) * S + D
    return O


def gated_streaming_rows(Q, K, V, log_a, geo, rows):
    """Gated streaming decode of the recent block: cached U^(n) of keys rescaled to the boundary, S_t = a_t S_{t-1} + Z_t,
    g_t = a_t g_{t-1}, ȳ_t = φ_tᵀ(g_t U_type + S_t)."""
    Q = np.asarray(Q, dtype=np.float64); K = np.asarray(K, dtype=np.float64); V = np.asarray(V, dtype=np.float64)
    a = np.exp(np.asarray(log_a, dtype=np.float64))
    lam = np.cumsum(np.asarray(log_a, dtype=np.float64))
    r, p = Q.shape[1], V.shape[1]
    F = np.zeros((geo.P, r, p))
    for t in range(geo.n):
        F[_profile(t, geo)] += np.exp(lam[geo.n - 1] - lam[t]) * np.outer(K[t], V[t])
    U = tabulate(F, geo)
    want = set(int(t) for t in rows)
    out, S, g = {}, np.zeros((r, p)), 1.0
    for t in range(geo.n, geo.T):
        S = a[t] * S + np.outer(K[t], V[t])
        g = a[t] * g
        if t in want:
            out[t] = Q[t] @ (g * U[_type(t, geo)] + S)
    return out
