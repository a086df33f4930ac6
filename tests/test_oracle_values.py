"""Pins for the oracle's values and gradients: special cases, linearity, finite differences,
and agreement between the dense definition and the paper's chunkwise equations."""
import numpy as np
import pytest

from oracle import chunkwise_ref as cw
from oracle import smat_oracle as so


def _rand(T, r, p, seed):
    g = np.random.default_rng(seed)
    return (g.standard_normal((T, r)) / np.sqrt(r), g.standard_normal((T, r)) / np.sqrt(r),
            g.standard_normal((T, p)), g.standard_normal((T, p)))


def _close(a, b, tol=1e-11):
    scale = max(1.0, float(np.max(np.abs(b))))
    assert float(np.max(np.abs(a - b))) <= tol * scale


# ---- special cases that reduce to textbook formulas ----------------------------------
def test_d1_equals_prefix_sum_linear_attention():
    T, r, p = 96, 8, 5
    Q, K, V, _ = _rand(T, r, p, 1)
    O = so.forward_dense(Q, K, V, so.dense_mask(T, 8, 1))
    S = np.zeros((r, p))
    for t in range(T):
        S += np.outer(K[t], V[t])            # running sum of k v^T
        _close(O[t], Q[t] @ S)


def test_d2_equals_bucketed_linear_attention():
    # d = 2: a hyperplane is a single point, so a recent query reads the bucket of distant
    # keys whose position is congruent to its own type (remark on d = 2 in the paper)
    T, c, r, p = 160, 8, 6, 4
    Q, K, V, _ = _rand(T, r, p, 2)
    geo = so.geometry(T, c, 2)
    q, n = geo.q, geo.n
    O = so.forward_dense(Q, K, V, so.dense_mask(T, c, 2))
    for t in range(T):
        acc = np.zeros(p)
        lo = 0 if t < n else n
        for s in range(lo, t + 1):
            acc += (Q[t] @ K[s]) * V[s]
        if t >= n:
            bucket = (t - n + 1) % q
            for s in range(n):
                if s % q == bucket:
                    acc += (Q[t] @ K[s]) * V[s]
        _close(O[t], acc)


def test_output_is_linear_in_the_mask():
    T, c, d = 128, 8, 3
    Q, K, V, _ = _rand(T, 8, 8, 3)
    geo = so.geometry(T, c, d)
    M = so.dense_mask(T, c, d).astype(np.float64)
    causal = M.copy()
    causal[geo.n:, :geo.n] = 0
    longr = M - causal
    _close(so.forward_dense(Q, K, V, M), so.forward_dense(Q, K, V, causal) + so.forward_dense(Q, K, V, longr))


def test_naive_triple_loop_on_a_tiny_case():
    T, c, d, q = 24, 2, 3, 2
    Q, K, V, dO = _rand(T, 3, 2, 4)
    M = so.dense_mask(T, c, d, q)
    O = so.forward_dense(Q, K, V, M)
    dQ, dK, dV = so.backward_dense(Q, K, V, dO, M)
    O2 = np.zeros_like(O); dQ2 = np.zeros_like(dQ); dK2 = np.zeros_like(dK); dV2 = np.zeros_like(dV)
    for t in range(T):
        for s in range(T):
            if M[t, s]:
                w = float(Q[t] @ K[s])
                O2[t] += w * V[s]
                gw = float(dO[t] @ V[s])
                dQ2[t] += gw * K[s]
                dK2[s] += gw * Q[t]
                dV2[s] += w * dO[t]
    _close(O, O2); _close(dQ, dQ2); _close(dK, dK2); _close(dV, dV2)


# ---- gradients -----------------------------------------------------------------------
@pytest.mark.parametrize("T,c,d,q", [(64, 4, 3, 3), (48, 4, 2, None), (40, 4, 1, None)])
def test_gradients_by_central_differences(T, c, d, q):
    # O is linear in each of Q, K, V, so a central difference is exact up to rounding
    Q, K, V, dO = _rand(T, 5, 4, 5)
    M = so.dense_mask(T, c, d, q)
    dQ, dK, dV = so.backward_dense(Q, K, V, dO, M)
    g = np.random.default_rng(6)
    loss = lambda q_, k_, v_: float(np.sum(dO * so.forward_dense(q_, k_, v_, M)))
    h = 0.5
    for name, X, dX in (("Q", Q, dQ), ("K", K, dK), ("V", V, dV)):
        E = g.standard_normal(X.shape)
        args_p = {"Q": Q, "K": K, "V": V}; args_m = dict(args_p)
        args_p[name] = X + h * E; args_m[name] = X - h * E
        fd = (loss(args_p["Q"], args_p["K"], args_p["V"]) - loss(args_m["Q"], args_m["K"], args_m["V"])) / (2 * h)
        assert abs(fd - float(np.sum(dX * E))) <= 1e-9 * max(1.0, abs(fd))


def test_adjoint_identities():
    T, c, d = 96, 8, 3
    Q, K, V, dO = _rand(T, 6, 7, 7)
    M = so.dense_mask(T, c, d)
    O = so.forward_dense(Q, K, V, M)
    dQ, dK, dV = so.backward_dense(Q, K, V, dO, M)
    ref = float(np.sum(dO * O))
    for X, dX in ((Q, dQ), (K, dK), (V, dV)):       # Euler: a degree-1 homogeneous map
        assert abs(float(np.sum(X * dX)) - ref) <= 1e-10 * max(1.0, abs(ref))


# ---- the paper's chunkwise equations give the same numbers --------------------------
CASES = [(128, 8, 1, None), (128, 8, 2, None), (192, 8, 3, None), (256, 16, 3, 5), (256, 8, 4, 3), (100, 8, 3, 3)]


@pytest.mark.parametrize("T,c,d,q", CASES)
def test_algorithm1_matches_the_dense_definition(T, c, d, q):
    Q, K, V, _ = _rand(T, 6, 5, 8)
    geo = so.geometry(T, c, d, q)
    _close(cw.forward(Q, K, V, geo), so.forward_dense(Q, K, V, so.dense_mask(T, c, d, q)))


@pytest.mark.parametrize("T,c,d,q", CASES)
def test_adjoint_equations_match_the_dense_gradients(T, c, d, q):
    Q, K, V, dO = _rand(T, 6, 5, 9)
    geo = so.geometry(T, c, d, q)
    ref = so.backward_dense(Q, K, V, dO, so.dense_mask(T, c, d, q))
    got = cw.backward(Q, K, V, dO, geo)
    for a, b in zip(got, ref):
        _close(a, b)


def test_streaming_evaluation_matches_the_dense_definition():
    T, c, d = 192, 8, 3
    Q, K, V, _ = _rand(T, 6, 5, 10)
    geo = so.geometry(T, c, d)
    O = so.forward_dense(Q, K, V, so.dense_mask(T, c, d))
    rows = list(range(geo.n, T, 7)) + [T - 1]
    got = cw.streaming_rows(Q, K, V, geo, rows)
    for t in rows:
        _close(got[t], O[t], 1e-12)


def test_chunk_size_invariance_at_fixed_boundary():
    # T a multiple of 2c for every c below, so n = T/2 and the mask is the same
    T, d = 512, 2
    Q, K, V, dO = _rand(T, 8, 8, 11)
    outs = []
    for c in (16, 32, 64, 128):
        geo = so.geometry(T, c, d)
        assert geo.n == 256
        outs.append((cw.forward(Q, K, V, geo),) + cw.backward(Q, K, V, dO, geo))
    for other in outs[1:]:
        for a, b in zip(other, outs[0]):
            _close(a, b)
    _close(outs[0][0], so.forward_dense(Q, K, V, so.dense_mask(T, 64, d)))


def test_tabulation_conserves_mass_per_direction():
    # for a fixed direction every point lies on exactly one hyperplane: Σ_b U_{a,b} = Σ_x F_x = Σ distant D_b
    T, c, d, q = 256, 8, 4, 3
    Q, K, V, _ = _rand(T, 4, 4, 12)
    geo = so.geometry(T, c, d, q)
    _, tab = cw.forward(Q, K, V, geo, return_tables=True)
    total = tab["F"].sum(axis=0)
    _close(tab["D"][: geo.n // c].sum(axis=0), total)
    U = tab["U"].reshape(geo.A, geo.q, *total.shape)
    for a in range(geo.A):
        _close(U[a].sum(axis=0), total)
    # tabulation equals multiplication by the explicit incidence matrix
    C = so.incidence_matrix(geo).astype(np.float64)
    _close(tab["U"].reshape(geo.B, -1), C @ tab["F"].reshape(geo.P, -1))
    Ubar = np.random.default_rng(0).standard_normal(tab["U"].shape)
    _close(cw.tabulate_transpose(Ubar, geo).reshape(geo.P, -1), C.T @ Ubar.reshape(geo.B, -1))


# ---- sampled rows / columns (what the large configurations use) ---------------------
def test_sampled_rows_and_columns_match_the_dense_results():
    T, c, d = 256, 16, 3
    Q, K, V, dO = _rand(T, 6, 5, 13)
    geo = so.geometry(T, c, d)
    M = so.dense_mask(T, c, d)
    O = so.forward_dense(Q, K, V, M)
    dQ, dK, dV = so.backward_dense(Q, K, V, dO, M)
    idx = [0, 1, geo.n - 1, geo.n, geo.n + 1, 200, T - 1]
    _close(so.forward_rows(Q, K, V, geo, idx), O[idx])
    _close(so.dq_rows(Q, K, V, dO, geo, idx), dQ[idx])
    gk, gv = so.dkdv_cols(Q, K, V, dO, geo, idx)
    _close(gk, dK[idx]); _close(gv, dV[idx])
