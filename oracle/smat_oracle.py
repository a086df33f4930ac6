"""Dense-mask fp64 oracle for hard-routing SMat-Attention.  TEST INFRASTRUCTURE ONLY.

This module is the definition written out: it builds the structured causal mask
M^(d) entry by entry and evaluates O = (M ⊙ QKᵀ) V and its gradients with plain
numpy in float64.  It is slow on purpose, contains no chunking, no tables and no
code shared with the CUDA library, and must only be imported by the tests, the
smoke check and the benchmark's CPU-baseline leg.

What follows which passage of the paper
---------------------------------------
* block form  M = [[L_n, 0], [G, L_m]]                     -> Eq. (blockform), Sec. 3
* hyperplanes H_{a,b} = {x : aᵀx = b} over F_q^{d-1}, count B -> Eq. (Bcount)
* G_ij = 1{prof(j) ∈ H_type(i)}                             -> Eq. (Gdef)
* positional assignment prof / type                         -> Sec. 3, "positional" item
* n = c·floor(T / 2c)                                       -> Sec. 3.1, causal branch
* d = 1: B = 1, G all ones, M = L_T                         -> Sec. 3, "Scaling with sequence length"
* output without feature map / normaliser: O = (M ⊙ QKᵀ)V   -> Eq. (augmented-attention-output)
  with φ = ψ = identity and the division left out

Readings taken where the paper is silent:
  R1  q = smallest prime with q^d >= n   (the paper only says q = Θ(n^{1/d}); this rule
      reproduces the decode-cache sizes printed in the end-to-end cost table)
  R2  prof digits are little-endian: x_1 is the least significant base-q digit of t mod q^{d-1}
  R3  type(i) = i mod B with the paper's 1-based i, i.e. the first recent token has type 1 mod B
  R4  type h = dir·q + b; directions ordered by the position g of their leading 1
      (g = 1 first), and inside a group by the tail (a_{g+1}, …, a_D) read as a
      little-endian base-q integer
  R5  T < 2c gives n = 0 and M = L_T for every d

Parity status: every function here is pinned by tests/test_oracle_*.py against closed
forms, theorem statements, brute force and printed values; the *bit order* choices
R2-R4 cannot be compared with the authors' code (absent) and are "parity unpinned"
in that narrow sense only — no stated property of the method depends on them.
"""
from __future__ import annotations

import itertools
from dataclasses import dataclass

import numpy as np


# --------------------------------------------------------------------------- geometry
def is_prime(v: int) -> bool:
    if v < 2:
        return False
    f = 2
    while f * f <= v:
        if v % f == 0:
            return False
        f += 1
    return True


def field_size(n: int, d: int) -> int:
    """Reading R1: the smallest prime q with q**d >= n (integer arithmetic only)."""
    q = 2
    while not (is_prime(q) and q ** d >= n):
        q += 1
    return q


@dataclass(frozen=True)
class Geometry:
    T: int
    c: int
    d: int
    n: int          # distant tokens
    m: int          # recent tokens
    q: int          # field size (0 when the long-range block is all ones)
    D: int          # ambient dimension d-1
    P: int          # number of profile cells q^(d-1)
    A: int          # number of normalised directions
    B: int          # number of types (hyperplanes)
    nnzC: int       # nonzeros of the incidence matrix = B q^(d-2)
    dense_G: bool   # True when G is all ones (d = 1)
    conditions_met: bool  # P <= n and 2B <= m (Sec. 3, scaling paragraph)


def geometry(T: int, c: int, d: int, q: int | None = None) -> Geometry:
    """Sizes of the construction (Sec. 3 and Sec. 3.1)."""
    if T < 1 or c < 1 or d < 1:
        raise ValueError("T, c, d must be positive")
    n = c * (T // (2 * c))
    m = T - n
    if d == 1 or n == 0:
        # d = 1: a single point and a single hyperplane that contains it; n = 0: no distant block
        return Geometry(T, c, d, n, m, 0, 0, 1, 1, 1, 1, True, True)
    if q is None:
        q = field_size(n, d)
    if not is_prime(q):
        raise ValueError("q must be prime")
    D = d - 1
    P = q ** D
    A = (P - 1) // (q - 1)
    B = q * A
    assert B == q * (q ** D - 1) // (q - 1)
    return Geometry(T, c, d, n, m, q, D, P, A, B, B * q ** (D - 1), False, (P <= n and 2 * B <= m))


def directions(q: int, D: int) -> list[tuple[int, ...]]:
    """All nonzero a ∈ F_q^D whose first nonzero coordinate is 1, in the order of reading R4."""
    out = []
    for g in range(1, D + 1):                       # position of the leading one (1-based)
        free = D - g                                 # coordinates after it are free
        for tail in range(q ** free):
            a = [0] * D
            a[g - 1] = 1
            v = tail
            for k in range(free):                    # little-endian digits of the tail
                a[g + k] = v % q
                v //= q
            out.append(tuple(a))
    return out


def prof(t: int, geo: Geometry) -> tuple[int, ...]:
    """Profile of the distant token t (0-based, t < n): base-q digits of t mod P (R2)."""
    v = t % geo.P
    x = []
    for _ in range(geo.D):
        x.append(v % geo.q)
        v //= geo.q
    return tuple(x)


def type_index(t: int, geo: Geometry) -> int:
    """Type of the recent token t (0-based, t >= n): the paper's i = t - n + 1, type = i mod B (R3)."""
    return (t - geo.n + 1) % geo.B


def type_pair(h: int, geo: Geometry) -> tuple[tuple[int, ...], int]:
    """(a, b) of type h under R4."""
    dirs = directions(geo.q, geo.D)
    return dirs[h // geo.q], h % geo.q


def on_hyperplane(x: tuple[int, ...], a: tuple[int, ...], b: int, q: int) -> bool:
    return sum(ai * xi for ai, xi in zip(a, x)) % q == b


def incidence_matrix(geo: Geometry) -> np.ndarray:
    """C[h, x] = 1{x ∈ H_h} with x indexed by its little-endian integer value (Eq. C)."""
    if geo.dense_G:
        return np.ones((1, 1), dtype=np.uint8)
    C = np.zeros((geo.B, geo.P), dtype=np.uint8)
    dirs = directions(geo.q, geo.D)
    pts = [prof(v, geo) for v in range(geo.P)]
    for h in range(geo.B):
        a, b = dirs[h // geo.q], h % geo.q
        for v, x in enumerate(pts):
            if on_hyperplane(x, a, b, geo.q):
                C[h, v] = 1
    return C


# --------------------------------------------------------------------------- mask
def mask_row(t: int, geo: Geometry) -> np.ndarray:
    """Row t of M^(d) from the definition (Eq. blockform, Eq. Gdef)."""
    row = np.zeros(geo.T, dtype=np.uint8)
    if t < geo.n:
        row[: t + 1] = 1
        return row
    row[geo.n : t + 1] = 1
    if geo.dense_G:
        row[: geo.n] = 1
        return row
    a, b = type_pair(type_index(t, geo), geo)
    s = np.arange(geo.n, dtype=np.int64) % geo.P
    acc = np.zeros(geo.n, dtype=np.int64)
    for ell in range(geo.D):
        acc += a[ell] * (s % geo.q)
        s //= geo.q
    row[: geo.n] = (acc % geo.q) == b
    return row


def mask_col(s: int, geo: Geometry) -> np.ndarray:
    """Column s of M^(d) from the definition."""
    col = np.zeros(geo.T, dtype=np.uint8)
    if s >= geo.n:
        col[s:] = 1
        return col
    col[s : geo.n] = 1
    if geo.dense_G:
        col[geo.n :] = 1
        return col
    x = prof(s, geo)
    dirs = directions(geo.q, geo.D)
    dots = np.array([sum(ai * xi for ai, xi in zip(a, x)) % geo.q for a in dirs], dtype=np.int64)
    h = (np.arange(geo.n, geo.T, dtype=np.int64) - geo.n + 1) % geo.B
    col[geo.n :] = dots[h // geo.q] == (h % geo.q)
    return col


# --------------------------------------------------------------------------- user-supplied routing
def routed_mask_row(t: int, geo: Geometry, prof_cells, types) -> np.ndarray:
    """Row t of the mask when the assignment is given explicitly (Sec. 3, "construction of G": any maps prof, type give
    G_ij = 1{prof(j) ∈ H_type(i)}, Eq. Gdef).  prof_cells[s] is the packed cell (little-endian base-q integer) of
    distant token s, types[i] the type of recent token n + i; an entry outside its range belongs to no cell / no type
    and contributes no long-range edge.  The two causal blocks do not depend on the assignment."""
    row = np.zeros(geo.T, dtype=np.uint8)
    if t < geo.n:
        row[: t + 1] = 1
        return row
    row[geo.n : t + 1] = 1
    if geo.dense_G:
        row[: geo.n] = 1
        return row
    h = int(types[t - geo.n])
    if not 0 <= h < geo.B:
        return row
    a, b = type_pair(h, geo)
    cells = np.asarray(prof_cells, dtype=np.int64)
    v = cells.copy()
    acc = np.zeros(geo.n, dtype=np.int64)
    for ell in range(geo.D):
        acc += a[ell] * (v % geo.q)
        v //= geo.q
    row[: geo.n] = ((acc % geo.q) == b) & (cells >= 0) & (cells < geo.P)
    return row


def routed_mask_col(s: int, geo: Geometry, prof_cells, types) -> np.ndarray:
    """Column s of the mask under an explicit assignment."""
    col = np.zeros(geo.T, dtype=np.uint8)
    if s >= geo.n:
        col[s:] = 1
        return col
    col[s : geo.n] = 1
    if geo.dense_G:
        col[geo.n :] = 1
        return col
    cell = int(prof_cells[s])
    if not 0 <= cell < geo.P:
        return col
    x = prof(cell, geo)                     # digits of the cell itself (prof() reduces its argument mod P)
    dirs = directions(geo.q, geo.D)
    dots = np.array([sum(ai * xi for ai, xi in zip(a, x)) % geo.q for a in dirs], dtype=np.int64)
    h = np.asarray(types, dtype=np.int64)
    ok = (h >= 0) & (h < geo.B)
    hh = np.where(ok, h, 0)
    col[geo.n :] = ok & (dots[hh // geo.q] == (hh % geo.q))
    return col


def routed_dense_mask(geo: Geometry, prof_cells, types) -> np.ndarray:
    return np.stack([routed_mask_row(t, geo, prof_cells, types) for t in range(geo.T)])


def positional_assignment(geo: Geometry):
    """The paper's positional prof / type as explicit arrays (packed cells, types)."""
    if geo.dense_G:
        return np.zeros(geo.n, dtype=np.int32), np.zeros(geo.m, dtype=np.int32)
    cells = (np.arange(geo.n, dtype=np.int64) % geo.P).astype(np.int32)
    types = np.array([type_index(t, geo) for t in range(geo.n, geo.T)], dtype=np.int32)
    return cells, types


def type_through_cell(geo: Geometry, direction_index: int, cell: int) -> int:
    """The content-based type of Sec. 3: the hyperplane with direction number `direction_index` that passes through
    `cell`, i.e. H_{a, aᵀu} for u the digits of the cell."""
    a = directions(geo.q, geo.D)[direction_index]
    u = prof(cell, geo)
    return direction_index * geo.q + sum(ai * ui for ai, ui in zip(a, u)) % geo.q


def routed_forward_rows(Q, K, V, geo: Geometry, prof_cells, types, rows):
    Q = np.asarray(Q, dtype=np.float64); K = np.asarray(K, dtype=np.float64); V = np.asarray(V, dtype=np.float64)
    out = np.empty((len(rows), V.shape[1]), dtype=np.float64)
    for k, t in enumerate(rows):
        out[k] = (routed_mask_row(int(t), geo, prof_cells, types) * (K @ Q[int(t)])) @ V
    return out


def routed_dq_rows(Q, K, V, dO, geo: Geometry, prof_cells, types, rows):
    K = np.asarray(K, dtype=np.float64); V = np.asarray(V, dtype=np.float64); dO = np.asarray(dO, dtype=np.float64)
    out = np.empty((len(rows), K.shape[1]), dtype=np.float64)
    for k, t in enumerate(rows):
        out[k] = (routed_mask_row(int(t), geo, prof_cells, types) * (V @ dO[int(t)])) @ K
    return out


def routed_dkdv_cols(Q, K, V, dO, geo: Geometry, prof_cells, types, cols):
    Q = np.asarray(Q, dtype=np.float64); K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64); dO = np.asarray(dO, dtype=np.float64)
    dK = np.empty((len(cols), K.shape[1]), dtype=np.float64)
    dV = np.empty((len(cols), V.shape[1]), dtype=np.float64)
    for k, s in enumerate(cols):
        mc = routed_mask_col(int(s), geo, prof_cells, types).astype(np.float64)
        dK[k] = (mc * (dO @ V[int(s)])) @ Q
        dV[k] = (mc * (Q @ K[int(s)])) @ dO
    return dK, dV


def dense_mask(T: int, c: int, d: int, q: int | None = None) -> np.ndarray:
    """The whole mask as a uint8 [T, T] array, one row at a time."""
    geo = geometry(T, c, d, q)
    return np.stack([mask_row(t, geo) for t in range(T)])


def routing_tables(geo: Geometry):
    """prof as packed integers (t mod P) with digits, type per recent token, (a, b) per type."""
    if geo.dense_G:
        return (np.zeros((geo.n, 0), dtype=np.int32), np.zeros(geo.m, dtype=np.int32),
                np.zeros((1, 1), dtype=np.int32))
    prof_digits = np.array([prof(t, geo) for t in range(geo.n)], dtype=np.int32).reshape(geo.n, geo.D)
    types = np.array([type_index(t, geo) for t in range(geo.n, geo.T)], dtype=np.int32)
    dirs = directions(geo.q, geo.D)
    ab = np.array([list(dirs[h // geo.q]) + [h % geo.q] for h in range(geo.B)], dtype=np.int32)
    return prof_digits, types, ab


# --------------------------------------------------------------------------- values
def forward_dense(Q, K, V, M):
    """O = (M ⊙ QKᵀ) V in float64 for one head."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    return (M * (Q @ K.T)) @ V


def backward_dense(Q, K, V, dO, M):
    """Gradients of <dO, O> with respect to Q, K, V in float64 for one head."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    dP = M * (dO @ V.T)          # gradient w.r.t. the masked scores
    dQ = dP @ K
    dK = dP.T @ Q
    dV = (M * (Q @ K.T)).T @ dO
    return dQ, dK, dV


def forward_rows(Q, K, V, geo: Geometry, rows):
    """Selected rows of O, each from its own explicitly built mask row."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    out = np.empty((len(rows), V.shape[1]), dtype=np.float64)
    for k, t in enumerate(rows):
        w = mask_row(int(t), geo) * (K @ Q[int(t)])
        out[k] = w @ V
    return out


def dq_rows(Q, K, V, dO, geo: Geometry, rows):
    """Selected rows of dQ."""
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    out = np.empty((len(rows), K.shape[1]), dtype=np.float64)
    for k, t in enumerate(rows):
        w = mask_row(int(t), geo) * (V @ dO[int(t)])
        out[k] = w @ K
    return out


def dkdv_cols(Q, K, V, dO, geo: Geometry, cols):
    """Selected rows of dK and dV (each is a column of the mask)."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    dO = np.asarray(dO, dtype=np.float64)
    dK = np.empty((len(cols), K.shape[1]), dtype=np.float64)
    dV = np.empty((len(cols), V.shape[1]), dtype=np.float64)
    for k, s in enumerate(cols):
        mc = mask_col(int(s), geo).astype(np.float64)
        dK[k] = (mc * (dO @ V[int(s)])) @ Q
        dV[k] = (mc * (Q @ K[int(s)])) @ dO
    return dK, dV


# --------------------------------------------------------------------------- gated mask (Sec. 3.2)
def decay_matrix(log_a) -> np.ndarray:
    """exp(λ_t - λ_s) for s <= t (0 elsewhere), λ_t = Σ_{k<=t} log a_k, from per-token log-gates log a_k <= 0
    (Eq. gated).  Every factor is formed as the exponential of a difference, so nothing overflows."""
    lam = np.cumsum(np.asarray(log_a, dtype=np.float64))
    diff = lam[:, None] - lam[None, :]
    return np.where(np.tril(np.ones_like(diff, dtype=bool)), np.exp(np.minimum(diff, 0.0)), 0.0)


def gated_forward_dense(Q, K, V, M, log_a):
    """O = ((M ⊙ decay) ⊙ QKᵀ) V: the binary mask replaced by the continuous mask of Eq. gated."""
    return forward_dense(Q, K, V, np.asarray(M, dtype=np.float64) * decay_matrix(log_a))


def gated_backward_dense(Q, K, V, dO, M, log_a):
    """Gradients of <dO, O> with respect to Q, K, V and the log-gates.  With W = M ⊙ decay ⊙ (dO Vᵀ) ⊙ (QKᵀ) (the
    contribution of every edge), ∂/∂λ_t is the sum of W over row t minus the sum over column t, and log a_k enters
    every λ_t with t >= k."""
    Q = np.asarray(Q, dtype=np.float64); K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64); dO = np.asarray(dO, dtype=np.float64)
    Mt = np.asarray(M, dtype=np.float64) * decay_matrix(log_a)
    dQ, dK, dV = backward_dense(Q, K, V, dO, Mt)
    W = Mt * (dO @ V.T) * (Q @ K.T)
    dlam = W.sum(axis=1) - W.sum(axis=0)
    dlog_a = np.cumsum(dlam[::-1])[::-1]
    return dQ, dK, dV, dlog_a


def gated_forward_rows(Q, K, V, geo: Geometry, log_a, rows):
    Q = np.asarray(Q, dtype=np.float64); K = np.asarray(K, dtype=np.float64); V = np.asarray(V, dtype=np.float64)
    lam = np.cumsum(np.asarray(log_a, dtype=np.float64))
    out = np.empty((len(rows), V.shape[1]), dtype=np.float64)
    for k, t in enumerate(rows):
        t = int(t)
        w = mask_row(t, geo) * np.exp(np.minimum(lam[t] - lam, 0.0)) * (K @ Q[t])
        out[k] = w @ V
    return out


# --------------------------------------------------------------------------- normalised output (Sec. 2)
def normalized_forward_dense(Q, K, V, M):
    """o_i = ȳ_{1:d_v} / ȳ_p with the augmented value v̄_j = [v_j; 1] (Eq. augmented-kv-state,
    Eq. augmented-attention-output): numerator (M ⊙ QKᵀ)V, normaliser (M ⊙ QKᵀ)1.  Returns (O, normaliser).
    Requires positive normalisers (non-negative features)."""
    Q = np.asarray(Q, dtype=np.float64); K = np.asarray(K, dtype=np.float64); V = np.asarray(V, dtype=np.float64)
    W = np.asarray(M, dtype=np.float64) * (Q @ K.T)
    den = W.sum(axis=1)
    return (W @ V) / den[:, None], den


def normalized_backward_dense(Q, K, V, dO, M):
    """Gradients of <dO, O> for the normalised output, through the final division: with Y = W V and z = W 1,
    dY = dO / z and dz = -Σ_c dO_c O_c / z; then the linear part with the augmented upstream [dY, dz]."""
    Q = np.asarray(Q, dtype=np.float64); K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64); dO = np.asarray(dO, dtype=np.float64)
    O, den = normalized_forward_dense(Q, K, V, M)
    dY = dO / den[:, None]
    dz = -np.sum(dO * O, axis=1) / den
    Vbar = np.concatenate([V, np.ones((V.shape[0], 1))], axis=1)
    dQ, dK, dVbar = backward_dense(Q, K, Vbar, np.concatenate([dY, dz[:, None]], axis=1), M)
    return dQ, dK, dVbar[:, :-1]


def normalized_forward_rows(Q, K, V, geo: Geometry, rows):
    Q = np.asarray(Q, dtype=np.float64); K = np.asarray(K, dtype=np.float64); V = np.asarray(V, dtype=np.float64)
    out = np.empty((len(rows), V.shape[1]), dtype=np.float64)
    den = np.empty(len(rows), dtype=np.float64)
    for k, t in enumerate(rows):
        w = mask_row(int(t), geo) * (K @ Q[int(t)])
        den[k] = w.sum()
        out[k] = (w @ V) / den[k]
    return out, den


# --------------------------------------------------------------------------- VC dimension
def vc_dimension(M: np.ndarray, limit: int | None = None) -> int:
    """Brute-force VC dimension of the row supports of a 0/1 matrix (Sec. 2, "VC dimension of a mask").

    Level-wise search: a k-set of columns can be shattered only if all its (k-1)-subsets are.
    """
    M = np.asarray(M, dtype=np.uint8)
    rows = np.unique(M, axis=0)
    ncols = M.shape[1]

    def shattered(cols):
        sub = rows[:, list(cols)]
        weights = 1 << np.arange(len(cols))
        return len(np.unique(sub @ weights)) == (1 << len(cols))

    level = [(j,) for j in range(ncols) if shattered((j,))]
    k = 0
    while level:
        k += 1
        if limit is not None and k >= limit:
            return k
        prev = set(level)
        nxt = []
        for s in level:
            for j in range(s[-1] + 1, ncols):
                cand = s + (j,)
                if all(tuple(cand[:i] + cand[i + 1:]) in prev for i in range(len(cand))):
                    if shattered(cand):
                        nxt.append(cand)
        level = nxt
    return k


def set_is_shattered(row_fn, cols, candidate_rows) -> bool:
    """True when the given rows realise every subset of `cols` (used for the witness set J_*)."""
    seen = set()
    for t in candidate_rows:
        r = row_fn(int(t))
        seen.add(tuple(int(r[j]) for j in cols))
    return len(seen) == (1 << len(cols))
