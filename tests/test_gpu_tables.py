"""Whole profile and type tables of one head at benchmark size against the fp64 chunkwise restatement (itself pinned
to the dense oracle): every (slab, CTA, image) of the tabulation kernels is covered, not only the states that the
sampled output rows happen to read.  Also the per-tile incoming states of the tensor-core causal branch."""
import numpy as np
import pytest
import torch

from oracle import chunkwise_ref as cw
from oracle import smat_oracle as so
from paper_2609_36062_b200 import binding, synth
from tests.helpers import device_inputs, rel_err, to_numpy64

pytestmark = pytest.mark.gpu

F_TOL, U_TOL = 8e-3, 1.2e-2     # one bf16 rounding per stored entry; U of d = 4 carries up to three


def _reference_tables(w, host, head, geo, directions=None):
    K64, V64 = (synth.as_float64(w, host[x][head]) for x in ("k", "v"))
    F = np.zeros((geo.P, w.d_k, w.d_v))
    for x in range(geo.P):                                       # Eq. "schedule": pooled outer products per profile
        F[x] = K64[x:geo.n:geo.P].T @ V64[x:geo.n:geo.P]
    if directions is None:
        return F, cw.tabulate(F, geo), np.arange(geo.B)
    pts = cw._point_digits(geo)
    dirs = so.directions(geo.q, geo.D)
    rows, U = [], []
    for ai in directions:                                        # the same offset classes, for a subset of directions
        off = (pts @ np.asarray(dirs[ai], dtype=np.int64)) % geo.q
        for b in range(geo.q):
            rows.append(ai * geo.q + b)
            U.append(F[off == b].sum(axis=0))
    return F, np.stack(U), np.asarray(rows)


@pytest.mark.parametrize("name,head,ndirs", [("t16k_d4", 5, None), ("t64k_d3", 3, None), ("t64k_d4", 9, 20)])
def test_full_tables_of_one_head_at_benchmark_size(name, head, ndirs):
    w = synth.WORKLOADS[name]
    host, dev = device_inputs(w)
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype)
    plan.forward(dev["q"], dev["k"], dev["v"])
    plan.check_status()
    F, U, _ = plan.debug_tables()
    geo = so.geometry(w.T, w.chunk, w.d)
    directions = None
    if ndirs is not None:
        rng = np.random.default_rng(4)
        directions = sorted(set([0, geo.A - 1]) | set(int(v) for v in rng.choice(geo.A, ndirs, replace=False)))
    Fref, Uref, rows = _reference_tables(w, host, head, geo, directions)
    assert rel_err(to_numpy64(F[head]), Fref) <= F_TOL
    got = to_numpy64(U[head][torch.as_tensor(rows, device=U.device)])
    assert rel_err(got, Uref) <= U_TOL
    # per state, so that a wrong row cannot hide behind a larger neighbour
    scale = np.abs(Uref).reshape(len(rows), -1).max(axis=1)
    worst = np.abs(got - Uref).reshape(len(rows), -1).max(axis=1) / np.maximum(scale, 1e-30)
    assert worst.max() <= 2.5 * U_TOL, (int(rows[worst.argmax()]), float(worst.max()))


@pytest.mark.parametrize("d,T", [(1, 2048), (3, 4096)])
def test_per_tile_incoming_states_are_exported(d, T):
    w = synth.Workload("tiles", d, 1, 2, T, 128, 128, 128, "bf16", "normalised", 91)
    host, dev = device_inputs(w)
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, flags=binding.FLAG_PER_TILE_STATES)
    assert plan.uses_tensor_cores()
    plan.forward(dev["q"], dev["k"], dev["v"])
    plan.check_status()
    F, U, Sin = plan.debug_tables()
    geo = so.geometry(T, 128, d)
    Q64, K64, V64 = (synth.as_float64(w, host[x][1]) for x in ("q", "k", "v"))
    _, tab = cw.forward(Q64, K64, V64, geo, return_tables=True)
    ref = tab["Sin"].copy()
    if d == 1:                                                   # the scan carries U_0 = F_0 through the boundary
        ref[geo.n // 128:] += tab["U"][0]
        assert rel_err(to_numpy64(U[1]), tab["U"]) <= 8e-3
        assert rel_err(to_numpy64(F[1]), tab["F"]) <= 8e-3
    assert Sin.shape[1] == T // 128
    assert rel_err(to_numpy64(Sin[1]), ref) <= 8e-3
    # the two-level form has no per-tile table to export
    seg = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype)
    seg.forward(dev["q"], dev["k"], dev["v"])
    lib = binding.load_library()
    buf = torch.empty_like(Sin)
    assert lib.smat_debug_tables(seg.handle, seg._ws.data_ptr(), None, None, buf.data_ptr(), None) == 10
