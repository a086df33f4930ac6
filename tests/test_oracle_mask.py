"""Pins for the oracle's mask: Theorem 1, the two VC lemmas, the witness construction."""
import itertools

import numpy as np
import pytest

from oracle import smat_oracle as so
from paper_2609_36062_b200 import synth


@pytest.mark.parametrize("T,c,d,q", [(16, 1, 1, None), (64, 4, 2, None), (96, 4, 3, 3), (128, 8, 3, None),
                                     (128, 4, 4, 2), (200, 8, 2, None)])
def test_theorem1_causal_unit_diagonal_and_nnz_bounds(T, c, d, q):
    M = so.dense_mask(T, c, d, q)
    assert M.shape == (T, T) and set(np.unique(M)) <= {0, 1}
    assert (np.triu(M, 1) == 0).all()            # causal
    assert (np.diag(M) == 1).all()               # unit diagonal
    nnz = int(M.sum())
    assert T * T / 4 <= nnz <= T * (T + 1) // 2  # proof of Theorem 1, nnz bounds
    geo = so.geometry(T, c, d, q)
    n, m = geo.n, geo.m
    assert (M[:n, :n] == np.tril(np.ones((n, n), dtype=np.uint8))).all()
    assert (M[n:, n:] == np.tril(np.ones((m, m), dtype=np.uint8))).all()
    assert (M[:n, n:] == 0).all()


@pytest.mark.parametrize("T,c", [(2, 1), (16, 1), (64, 8), (100, 8)])
def test_d1_is_the_causal_mask(T, c):
    assert (so.dense_mask(T, c, 1) == np.tril(np.ones((T, T), dtype=np.uint8))).all()


def test_short_sequence_has_no_distant_block():
    assert (so.dense_mask(12, 8, 3) == np.tril(np.ones((12, 12), dtype=np.uint8))).all()


@pytest.mark.parametrize("T,c,d,q", [(100, 5, 2, 5), (108, 2, 3, 3), (128, 8, 4, 2), (250, 5, 3, 5)])
def test_exact_nnz_when_profiles_divide_n(T, c, d, q):
    geo = so.geometry(T, c, d, q)
    assert geo.n % geo.P == 0
    M = so.dense_mask(T, c, d, q)
    n, m = geo.n, geo.m
    # each hyperplane holds a 1/q share of the profile cells, hence of the distant tokens
    assert int(M.sum()) == n * (n + 1) // 2 + m * (m + 1) // 2 + m * n // q


def test_G_depends_only_on_type_and_profile():
    geo = so.geometry(256, 4, 3, 5)
    M = so.dense_mask(256, 4, 3, 5)
    C = so.incidence_matrix(geo)
    G = M[geo.n:, :geo.n]
    types = np.array([so.type_index(t, geo) for t in range(geo.n, geo.T)])
    profs = np.arange(geo.n) % geo.P
    assert (G == C[types][:, profs]).all()


def test_rows_and_columns_agree_with_the_dense_mask():
    for (T, c, d, q) in [(128, 8, 3, None), (128, 4, 4, 2), (64, 4, 1, None), (96, 8, 2, None)]:
        geo = so.geometry(T, c, d, q)
        M = so.dense_mask(T, c, d, q)
        for s in range(T):
            assert (so.mask_col(s, geo) == M[:, s]).all()


# ---- VC dimension -------------------------------------------------------------------
@pytest.mark.parametrize("T", [2, 3, 8, 20])
def test_lemma_lower_triangular_has_vc_one(T):
    assert so.vc_dimension(np.tril(np.ones((T, T), dtype=np.uint8))) == 1


def test_lemma_single_row_has_vc_zero():
    assert so.vc_dimension(np.ones((1, 1), dtype=np.uint8)) == 0


@pytest.mark.parametrize("q,D", [(2, 2), (3, 2), (2, 3), (5, 1), (3, 3)])
def test_lemma_affine_hyperplanes_have_vc_exactly_D(q, D):
    pts = list(itertools.product(range(q), repeat=D))
    rows = []
    for a in itertools.product(range(q), repeat=D):
        if not any(a):
            continue
        for b in range(q):
            rows.append([1 if sum(ai * xi for ai, xi in zip(a, x)) % q == b else 0 for x in pts])
    assert so.vc_dimension(np.array(rows, dtype=np.uint8)) == D


def test_vc_search_on_a_known_set_system():
    # all subsets of 3 points: VC 3;   intervals on a line of 6 points: VC 2
    full = np.array(list(itertools.product([0, 1], repeat=3)), dtype=np.uint8)
    assert so.vc_dimension(full) == 3
    iv = [[1 if lo <= j < hi else 0 for j in range(6)] for lo in range(7) for hi in range(lo, 7)]
    assert so.vc_dimension(np.array(iv, dtype=np.uint8)) == 2


# (T, c, d, q) -> (VC, nnz): brute force; the expected pairs were obtained independently while surveying the paper
@pytest.mark.parametrize("T,c,d,q,vc,nnz", [
    (16, 1, 1, None, 1, 136),
    (16, 1, 2, 3, 2, 93),
    (32, 2, 2, 5, 2, 323),
    (32, 1, 3, 2, 3, 400),
    (64, 1, 3, 3, 3, 1397),
    (64, 1, 4, 2, 4, 1568),
])
def test_theorem1_vc_dimension_equals_d(T, c, d, q, vc, nnz):
    M = so.dense_mask(T, c, d, q)
    assert int(M.sum()) == nnz
    geo = so.geometry(T, c, d, q)
    assert geo.conditions_met
    assert so.vc_dimension(M) == vc == d


def test_theorem1_vc_dimension_d3_q5():
    M = so.dense_mask(128, 1, 3, 5)
    assert int(M.sum()) == 4979
    assert so.vc_dimension(M) == 3


def _witness_is_shattered(geo):
    """The set J_* = {j_1..j_D, n+τ} of the lower-bound proof, realised by recent rows i in [1, 2B]."""
    D, q, n, B = geo.D, geo.q, geo.n, geo.B
    cols = [q ** ell for ell in range(D)]                 # prof = e_{ell+1} (0-based token index)
    for t, ell in zip(cols, range(D)):
        e = tuple(1 if k == ell else 0 for k in range(D))
        assert so.prof(t, geo) == e
    tau = B + 1                                           # every type occurs in [1, B] and in [B+1, 2B]
    cols.append(n + tau - 1)
    cand = range(n, n + 2 * B)
    return so.set_is_shattered(lambda t: so.mask_row(t, geo), cols, cand)


@pytest.mark.parametrize("name", ["small_d2", "t4k_d3", "t16k_d4", "t64k_d2", "t64k_d3", "t64k_d4", "t8k_d3_fwdbwd"])
def test_witness_set_is_shattered_on_every_workload(name):
    w = synth.WORKLOADS[name]
    geo = so.geometry(w.T, w.chunk, w.d)
    assert geo.conditions_met
    if geo.B > 1500:                                      # keep the CPU suite short: rows of the 2^d witness types only
        D, q, n, B = geo.D, geo.q, geo.n, geo.B
        dirs = so.directions(q, D)
        cols = [q ** ell for ell in range(D)] + [n + B]
        seen = set()
        for R in itertools.product([0, 1], repeat=D):
            if all(R):
                a, b = tuple([1] * D), 1
            else:
                a, b = tuple(1 - v for v in R), 0
            h = dirs.index(a) * q + b
            i_minus = h if h >= 1 else B
            for i in (i_minus, i_minus + B):
                row = so.mask_row(n + i - 1, geo)
                seen.add(tuple(int(row[j]) for j in cols))
        assert len(seen) == 2 ** d_of(geo)
    else:
        assert _witness_is_shattered(geo)


def d_of(geo):
    return geo.d


# ---- set_is_shattered itself: cases where the answer must be False ------------------------------------
def test_shattering_check_rejects_sets_that_are_not_shattered():
    # a hand-made set system: three columns, rows realise 7 of the 8 patterns
    rows = [r for r in itertools.product([0, 1], repeat=3) if r != (1, 0, 1)]
    table = np.array(rows, dtype=np.uint8)
    assert not so.set_is_shattered(lambda t: table[t], [0, 1, 2], range(len(rows)))
    assert so.set_is_shattered(lambda t: table[t], [0, 1], range(len(rows)))
    full = np.array(list(itertools.product([0, 1], repeat=3)), dtype=np.uint8)
    assert so.set_is_shattered(lambda t: full[t], [0, 1, 2], range(8))
    assert not so.set_is_shattered(lambda t: full[t], [0, 1, 2], range(7))      # one pattern's row withheld


@pytest.mark.parametrize("T,c,d,q", [(256, 4, 3, 5), (512, 64, 2, None), (1024, 16, 4, 3)])
def test_witness_set_needs_both_sides_of_tau_and_cannot_grow(T, c, d, q):
    """Lower-bound proof of Theorem 1: the last witness column n+τ separates recent rows before τ from rows after it.
    With only the first B recent rows (every type once, all before τ = B+1) that column is never set, so the witness
    set is NOT shattered; with 2B rows it is; and no set of d+1 columns is shattered by any rows (VC = d)."""
    geo = so.geometry(T, c, d, q)
    assert geo.conditions_met
    D, n, B = geo.D, geo.n, geo.B
    cols = [geo.q ** ell for ell in range(D)] + [n + B]
    row = lambda t: so.mask_row(t, geo)
    assert so.set_is_shattered(row, cols, range(n, n + 2 * B))
    assert not so.set_is_shattered(row, cols, range(n, n + B))          # no row lies on the far side of τ
    assert not so.set_is_shattered(row, cols, range(n + B, n + 2 * B))  # ... nor any on the near side
    assert so.set_is_shattered(row, cols[:-1], range(n, n + B))         # the D profile columns alone need one side
    # d+1 columns: the witness set plus any further column is not shattered by the whole mask (upper bound VC <= d)
    for extra in (0, geo.q + 1, n - 1, n, n + 2 * B - 1, T - 1):
        if extra in cols:
            continue
        assert not so.set_is_shattered(row, cols + [extra], range(T)), extra
