"""Pins for the oracle's user-supplied routing (explicit prof / type arrays, Sec. 3 "construction of G")."""
import numpy as np
import pytest

from oracle import smat_oracle as so


CASES = [(96, 4, 3, 3), (128, 8, 2, None), (128, 4, 4, 2), (200, 4, 3, 5)]


@pytest.mark.parametrize("T,c,d,q", CASES)
def test_positional_arrays_reproduce_the_positional_mask_bit_for_bit(T, c, d, q):
    geo = so.geometry(T, c, d, q)
    cells, types = so.positional_assignment(geo)
    assert np.array_equal(so.routed_dense_mask(geo, cells, types), so.dense_mask(T, c, d, q))


@pytest.mark.parametrize("T,c,d,q", CASES)
def test_G_is_the_incidence_matrix_indexed_by_the_two_maps(T, c, d, q):
    """Eq. Gdef with Eq. C: G = R C Eᵀ for ANY assignment, checked against the explicit incidence matrix."""
    geo = so.geometry(T, c, d, q)
    g = np.random.default_rng(T + d)
    cells = g.integers(0, geo.P, geo.n)
    types = g.integers(0, geo.B, geo.m)
    M = so.routed_dense_mask(geo, cells, types)
    C = so.incidence_matrix(geo)
    assert np.array_equal(M[geo.n:, :geo.n], C[types][:, cells])
    # the causal blocks do not depend on the assignment; rows and columns agree
    assert np.array_equal(M[:geo.n, :geo.n], np.tril(np.ones((geo.n, geo.n), dtype=np.uint8)))
    assert np.array_equal(M[geo.n:, geo.n:], np.tril(np.ones((geo.m, geo.m), dtype=np.uint8)))
    for s in range(0, T, 7):
        assert np.array_equal(so.routed_mask_col(s, geo, cells, types), M[:, s])


def test_out_of_range_entries_route_nowhere():
    geo = so.geometry(128, 4, 3, 3)
    g = np.random.default_rng(0)
    cells = g.integers(0, geo.P, geo.n)
    types = g.integers(0, geo.B, geo.m)
    cells[5], cells[11], types[3], types[9] = -1, geo.P, geo.B, -7
    M = so.routed_dense_mask(geo, cells, types)
    G = M[geo.n:, :geo.n]
    assert not G[:, 5].any() and not G[:, 11].any() and not G[3].any() and not G[9].any()
    for s in (5, 11, 20):
        assert np.array_equal(so.routed_mask_col(s, geo, cells, types), M[:, s])


@pytest.mark.parametrize("T,c,d,q", [(256, 4, 3, 5), (256, 8, 4, 3), (128, 4, 2, None)])
def test_content_based_type_sees_every_key_of_its_own_cell(T, c, d, q):
    """Content-based assignment: a query hashed to cell u with direction a gets the hyperplane H_{a, aᵀu} through its
    own cell, so it sees every distant key hashed to the same cell, and of the keys of any other cell either all or
    none; a cell is seen by the query iff it lies on that hyperplane, which holds for a 1/q share of the cells."""
    geo = so.geometry(T, c, d, q)
    g = np.random.default_rng(3)
    cells = g.integers(0, geo.P, geo.n)
    qcell = g.integers(0, geo.P, geo.m)
    qdir = g.integers(0, geo.A, geo.m)
    types = np.array([so.type_through_cell(geo, int(a), int(u)) for a, u in zip(qdir, qcell)])
    M = so.routed_dense_mask(geo, cells, types)
    G = M[geo.n:, :geo.n]
    for i in range(geo.m):
        assert G[i][cells == qcell[i]].all()
        seen_cells = {int(v) for v in cells[G[i] == 1]}
        for v in seen_cells:
            assert G[i][cells == v].all()
        a, b = so.type_pair(int(types[i]), geo)
        on_plane = [v for v in range(geo.P) if so.on_hyperplane(so.prof(v, geo), a, b, geo.q)]
        assert len(on_plane) == geo.P // geo.q and seen_cells <= set(on_plane)


def test_routed_rows_and_columns_match_the_dense_products():
    T, c, d, q = 160, 4, 3, 5
    geo = so.geometry(T, c, d, q)
    g = np.random.default_rng(9)
    Q, K = g.standard_normal((T, 6)), g.standard_normal((T, 6))
    V, dO = g.standard_normal((T, 5)), g.standard_normal((T, 5))
    cells = g.integers(0, geo.P, geo.n)
    types = g.integers(0, geo.B, geo.m)
    M = so.routed_dense_mask(geo, cells, types)
    O = so.forward_dense(Q, K, V, M)
    dQ, dK, dV = so.backward_dense(Q, K, V, dO, M)
    idx = [0, 3, geo.n - 1, geo.n, geo.n + 2, T - 1]
    assert np.allclose(so.routed_forward_rows(Q, K, V, geo, cells, types, idx), O[idx], atol=1e-12)
    assert np.allclose(so.routed_dq_rows(Q, K, V, dO, geo, cells, types, idx), dQ[idx], atol=1e-12)
    gk, gv = so.routed_dkdv_cols(Q, K, V, dO, geo, cells, types, idx)
    assert np.allclose(gk, dK[idx], atol=1e-12) and np.allclose(gv, dV[idx], atol=1e-12)
