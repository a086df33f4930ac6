"""Pins for the oracle's gated mask (Sec. 3.2, Eq. gated; Lemma "Gated SMat")."""
import numpy as np
import pytest

from oracle import chunkwise_ref as cw
from oracle import smat_oracle as so


def _rand(T, r, p, seed):
    g = np.random.default_rng(seed)
    return (g.standard_normal((T, r)) / np.sqrt(r), g.standard_normal((T, r)) / np.sqrt(r),
            g.standard_normal((T, p)), g.standard_normal((T, p)), np.log(g.uniform(0.6, 1.0, T)))


def _close(a, b, tol=1e-11):
    assert float(np.max(np.abs(a - b))) <= tol * max(1.0, float(np.max(np.abs(b))))


def test_unit_gates_give_the_binary_mask():
    T, c, d = 96, 8, 3
    Q, K, V, dO, _ = _rand(T, 6, 5, 1)
    M = so.dense_mask(T, c, d)
    zero = np.zeros(T)
    _close(so.gated_forward_dense(Q, K, V, M, zero), so.forward_dense(Q, K, V, M))
    g = so.gated_backward_dense(Q, K, V, dO, M, zero)
    for a, b in zip(g[:3], so.backward_dense(Q, K, V, dO, M)):
        _close(a, b)


def test_decay_is_the_product_of_the_gates_between_source_and_target():
    g = np.random.default_rng(2)
    a = g.uniform(0.3, 1.0, 12)
    D = so.decay_matrix(np.log(a))
    for t in range(12):
        for s in range(12):
            want = float(np.prod(a[s + 1 : t + 1])) if s <= t else 0.0
            assert abs(D[t, s] - want) <= 1e-14
    # entries lie in (0, 1] on and below the diagonal even when the cumulative sum is huge
    big = so.decay_matrix(np.full(4000, -1.0))
    assert np.isfinite(big).all() and big.max() == 1.0 and big[3999, 0] == 0.0


def test_d1_is_the_gated_linear_attention_recurrence():
    # d = 1: S_t = a_t S_{t-1} + k_t v_tᵀ,  o_t = q_tᵀ S_t
    T, r, p = 80, 6, 4
    Q, K, V, _, la = _rand(T, r, p, 3)
    O = so.gated_forward_dense(Q, K, V, so.dense_mask(T, 8, 1), la)
    S = np.zeros((r, p))
    for t in range(T):
        S = np.exp(la[t]) * S + np.outer(K[t], V[t])
        _close(O[t], Q[t] @ S)


def test_naive_loop_on_a_tiny_case():
    T, c, d, q = 24, 2, 3, 2
    Q, K, V, _, la = _rand(T, 3, 2, 4)
    M = so.dense_mask(T, c, d, q)
    O = so.gated_forward_dense(Q, K, V, M, la)
    a = np.exp(la)
    ref = np.zeros_like(O)
    for t in range(T):
        for s in range(t + 1):
            if M[t, s]:
                ref[t] += np.prod(a[s + 1 : t + 1]) * float(Q[t] @ K[s]) * V[s]
    _close(O, ref)


@pytest.mark.parametrize("T,c,d,q", [(64, 4, 3, 3), (48, 4, 2, None), (40, 4, 1, None)])
def test_gated_gradients_by_central_differences(T, c, d, q):
    Q, K, V, dO, la = _rand(T, 5, 4, 5)
    M = so.dense_mask(T, c, d, q)
    dQ, dK, dV, dla = so.gated_backward_dense(Q, K, V, dO, M, la)
    loss = lambda q_, k_, v_, l_: float(np.sum(dO * so.gated_forward_dense(q_, k_, v_, M, l_)))
    g = np.random.default_rng(6)
    for X, dX, pos in ((Q, dQ, 0), (K, dK, 1), (V, dV, 2)):      # multilinear: a central difference is exact
        E = g.standard_normal(X.shape)
        args_p, args_m = [Q, K, V, la], [Q, K, V, la]
        args_p[pos] = X + 0.5 * E; args_m[pos] = X - 0.5 * E
        fd = loss(*args_p) - loss(*args_m)
        assert abs(fd - float(np.sum(dX * E))) <= 1e-9 * max(1.0, abs(fd))
    E = g.standard_normal(T)
    h = 1e-5                                                       # the gates enter through exp: second-order accurate
    fd = (loss(Q, K, V, la + h * E) - loss(Q, K, V, la - h * E)) / (2 * h)
    assert abs(fd - float(np.sum(dla * E))) <= 1e-7 * max(1.0, abs(fd))
    # the gate gradient from the other gradients: dλ_t = q_t·dQ_t - k_t·dK_t, summed over t >= k
    dlam = np.sum(Q * dQ, axis=1) - np.sum(K * dK, axis=1)
    _close(np.cumsum(dlam[::-1])[::-1], dla, 1e-10)


@pytest.mark.parametrize("T,c,d,q", [(128, 8, 1, None), (128, 8, 2, None), (192, 8, 3, None), (256, 8, 4, 3), (100, 8, 3, 3)])
def test_gated_chunkwise_lemma_matches_the_dense_definition(T, c, d, q):
    Q, K, V, _, la = _rand(T, 6, 5, 8)
    geo = so.geometry(T, c, d, q)
    M = so.dense_mask(T, c, d, q)
    ref = so.gated_forward_dense(Q, K, V, M, la)
    _close(cw.gated_forward(Q, K, V, la, geo), ref)
    rows = list(range(geo.n, T, 5)) + [T - 1]
    got = cw.gated_streaming_rows(Q, K, V, la, geo, rows)
    for t in rows:
        _close(got[t], ref[t])
    _close(so.gated_forward_rows(Q, K, V, geo, la, rows), ref[rows])


def test_strong_decay_does_not_overflow_in_the_chunkwise_form():
    T, c, d = 256, 16, 3
    Q, K, V, _, _ = _rand(T, 4, 4, 9)
    la = np.full(T, np.log(1e-3))                                 # λ reaches -1768: exp(-λ) would overflow
    geo = so.geometry(T, c, d)
    out = cw.gated_forward(Q, K, V, la, geo)
    assert np.isfinite(out).all()
    _close(out, so.gated_forward_dense(Q, K, V, so.dense_mask(T, c, d), la))
