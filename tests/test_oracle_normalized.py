"""Pins for the oracle's normalised output (Sec. 2: augmented value [v; 1], one final division)."""
import numpy as np
import pytest

from oracle import smat_oracle as so


def _pos(T, r, p, seed):
    g = np.random.default_rng(seed)
    return (np.abs(g.standard_normal((T, r))) + 0.05, np.abs(g.standard_normal((T, r))) + 0.05,
            g.standard_normal((T, p)), g.standard_normal((T, p)))


@pytest.mark.parametrize("T,c,d,q", [(96, 8, 3, 3), (64, 4, 2, None), (48, 4, 1, None), (128, 4, 4, 2)])
def test_weights_of_a_row_sum_to_one(T, c, d, q):
    """Each output row is a convex combination of the values it sees: constant values come back unchanged, and the
    output stays inside the range of the values column by column."""
    Q, K, V, _ = _pos(T, 5, 4, 1)
    M = so.dense_mask(T, c, d, q)
    O, den = so.normalized_forward_dense(Q, K, np.full_like(V, 2.5), M)
    assert (den > 0).all() and np.allclose(O, 2.5, atol=1e-12)
    O, _ = so.normalized_forward_dense(Q, K, V, M)
    for t in range(T):
        seen = V[M[t] == 1]
        assert (O[t] <= seen.max(axis=0) + 1e-12).all() and (O[t] >= seen.min(axis=0) - 1e-12).all()


def test_scaling_the_queries_or_keys_changes_nothing():
    T, c, d = 80, 8, 3
    Q, K, V, _ = _pos(T, 6, 3, 2)
    M = so.dense_mask(T, c, d)
    O, den = so.normalized_forward_dense(Q, K, V, M)
    O2, den2 = so.normalized_forward_dense(3.0 * Q, 0.25 * K, V, M)
    assert np.allclose(O, O2, atol=1e-12) and np.allclose(den2, 0.75 * den, rtol=1e-12)


def test_d1_is_normalised_causal_linear_attention_by_prefix_sums():
    T, r, p = 72, 6, 4
    Q, K, V, _ = _pos(T, r, p, 3)
    O, den = so.normalized_forward_dense(Q, K, V, so.dense_mask(T, 8, 1))
    S, z = np.zeros((r, p)), np.zeros(r)
    for t in range(T):
        S += np.outer(K[t], V[t]); z += K[t]
        assert np.allclose(O[t], (Q[t] @ S) / (Q[t] @ z), atol=1e-12) and abs(den[t] - Q[t] @ z) <= 1e-12


def test_augmented_value_column_gives_the_normaliser():
    # the paper's form: one pass with v̄ = [v; 1]; the last column of ȳ is the normaliser
    T, c, d = 64, 4, 3
    Q, K, V, _ = _pos(T, 5, 3, 4)
    M = so.dense_mask(T, c, d, 3)
    Y = so.forward_dense(Q, K, np.concatenate([V, np.ones((T, 1))], axis=1), M)
    O, den = so.normalized_forward_dense(Q, K, V, M)
    assert np.allclose(Y[:, -1], den, atol=1e-12) and np.allclose(Y[:, :-1] / Y[:, -1:], O, atol=1e-12)


@pytest.mark.parametrize("T,c,d,q", [(64, 4, 3, 3), (48, 4, 2, None), (40, 4, 1, None)])
def test_normalised_gradients_by_central_differences(T, c, d, q):
    Q, K, V, dO = _pos(T, 5, 4, 5)
    M = so.dense_mask(T, c, d, q)
    grads = so.normalized_backward_dense(Q, K, V, dO, M)
    loss = lambda q_, k_, v_: float(np.sum(dO * so.normalized_forward_dense(q_, k_, v_, M)[0]))
    g = np.random.default_rng(6)
    for pos, (X, dX) in enumerate(zip((Q, K, V), grads)):
        E = g.standard_normal(X.shape)
        h = 1e-6
        ap, am = [Q, K, V], [Q, K, V]
        ap[pos] = X + h * E; am[pos] = X - h * E
        fd = (loss(*ap) - loss(*am)) / (2 * h)
        assert abs(fd - float(np.sum(dX * E))) <= 1e-6 * max(1.0, abs(fd))
    # the output does not change along the ray through Q, so the gradient is orthogonal to it (Euler, degree 0)
    assert abs(float(np.sum(Q * grads[0]))) <= 1e-9 * float(np.sum(np.abs(Q * grads[0])))


def test_sampled_rows_match_the_dense_result():
    T, c, d = 128, 8, 3
    Q, K, V, _ = _pos(T, 4, 3, 7)
    geo = so.geometry(T, c, d)
    O, den = so.normalized_forward_dense(Q, K, V, so.dense_mask(T, c, d))
    idx = [0, 5, geo.n - 1, geo.n, T - 1]
    o, z = so.normalized_forward_rows(Q, K, V, geo, idx)
    assert np.allclose(o, O[idx], atol=1e-12) and np.allclose(z, den[idx], atol=1e-12)
