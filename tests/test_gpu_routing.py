"""User-supplied routing on the GPU (smat_forward_routed / smat_backward_routed) against the fp64 oracle with the same
explicit prof / type arrays: positional arrays must reproduce the positional call bit for bit, a seeded random hash
(uniform, heavily skewed, with empty cells and out-of-range entries) must match the dense-mask products."""
import numpy as np
import pytest
import torch

from oracle import smat_oracle as so
from paper_2609_36062_b200 import binding, synth
from tests.helpers import TOL, device_inputs, rel_err, sample_tokens, to_numpy64

pytestmark = pytest.mark.gpu


def _assignment(w, geo, skew, drop=False):
    cells, types = [], []
    for h in range(w.bh):
        c = synth.hashed_cells(w, h, geo.n, geo.P, skew)
        qcell, qdir = synth.hashed_query_draws(w, h, geo.m, geo.P, geo.A)
        t = np.array([so.type_through_cell(geo, int(a), int(u)) for a, u in zip(qdir, qcell)], dtype=np.int32)
        if drop:                                                 # a few tokens that belong to no cell / no type
            c[3], c[geo.n // 2], t[1], t[geo.m - 1] = -1, geo.P, geo.B + 5, -2
        cells.append(c); types.append(t)
    return np.stack(cells), np.stack(types)


@pytest.mark.parametrize("d,T,c,dtype,q", [(2, 2048, 128, "bf16", 0), (3, 4096, 128, "bf16", 0), (4, 4096, 128, "bf16", 0),
                                           (3, 512, 32, "f32", 0), (4, 1024, 16, "f32", 3), (3, 4096, 128, "bf16", 37)])
def test_positional_arrays_reproduce_the_positional_call(d, T, c, dtype, q):
    dk = 128 if dtype == "bf16" else 64
    w = synth.Workload("pos", d, 1, 2, T, dk, dk, c, dtype, "normalised", 33)
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    geo = so.geometry(T, c, d, q or None)
    cells, types = so.positional_assignment(geo)
    prof = torch.from_numpy(np.tile(cells, (w.bh, 1))).int().cuda()
    typ = torch.from_numpy(np.tile(types, (w.bh, 1))).int().cuda()
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, q_override=q)
    a = plan.forward(dev["q"], dev["k"], dev["v"]).clone()
    ga = [x.clone() for x in plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])]
    b = plan.forward(dev["q"], dev["k"], dev["v"], prof=prof, type=typ)
    gb = plan.backward(dev["q"], dev["k"], dev["v"], dev["do"], prof=prof, type=typ)
    plan.check_status()
    assert torch.equal(a, b)                                     # same groups, same token order inside every group
    for x, y in zip(ga, gb):
        assert torch.equal(x, y)


@pytest.mark.parametrize("d,T,c,dtype,q,skew,drop", [
    (2, 2048, 128, "bf16", 0, 0.0, False), (3, 4096, 128, "bf16", 0, 0.0, True), (4, 4096, 128, "bf16", 0, 0.0, False),
    (3, 4096, 128, "bf16", 0, 1.2, False),      # heavy cells (hundreds of tokens) and many empty ones
    (4, 8192, 128, "bf16", 0, 1.0, True), (3, 4096, 128, "bf16", 37, 0.0, False),
    (3, 512, 32, "f32", 0, 0.8, True), (2, 384, 16, "f32", 0, 0.0, False), (4, 1024, 16, "f32", 3, 0.0, False),
])
def test_hashed_routing_matches_the_dense_oracle(d, T, c, dtype, q, skew, drop):
    dk = 128 if dtype == "bf16" else 64
    w = synth.Workload("hash", d, 1, 2, T, dk, dk, c, dtype, "normalised", 55 + d)
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    geo = so.geometry(T, c, d, q or None)
    cells, types = _assignment(w, geo, skew, drop)
    prof, typ = torch.from_numpy(cells).cuda(), torch.from_numpy(types).cuda()
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, q_override=q)
    O = plan.forward(dev["q"], dev["k"], dev["v"], prof=prof, type=typ)
    dQ, dK, dV = plan.backward(dev["q"], dev["k"], dev["v"], dev["do"], prof=prof, type=typ)
    plan.check_status()
    tol = TOL[dtype]
    for h in range(w.bh):
        Q64, K64, V64, G64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v", "do"))
        if T <= 1024:
            M = so.routed_dense_mask(geo, cells[h], types[h])
            assert rel_err(to_numpy64(O[0, h]), so.forward_dense(Q64, K64, V64, M)) <= tol
            for got, ref in zip((dQ, dK, dV), so.backward_dense(Q64, K64, V64, G64, M)):
                assert rel_err(to_numpy64(got[0, h]), ref) <= tol
        else:
            rows = sample_tokens(geo, 72, seed=h)
            heavy = np.bincount(cells[h][(cells[h] >= 0) & (cells[h] < geo.P)], minlength=geo.P).argmax()
            rows = sorted(set(rows) | set(np.nonzero(cells[h] == heavy)[0][:6].tolist()))   # keys of the heaviest cell
            assert rel_err(to_numpy64(O[0, h][rows]), so.routed_forward_rows(Q64, K64, V64, geo, cells[h], types[h], rows)) <= tol
            assert rel_err(to_numpy64(dQ[0, h][rows]), so.routed_dq_rows(Q64, K64, V64, G64, geo, cells[h], types[h], rows)) <= tol
            rk, rv = so.routed_dkdv_cols(Q64, K64, V64, G64, geo, cells[h], types[h], rows)
            assert rel_err(to_numpy64(dK[0, h][rows]), rk) <= tol
            assert rel_err(to_numpy64(dV[0, h][rows]), rv) <= tol


def test_routed_call_is_reproducible_and_validates_its_arguments():
    w = synth.Workload("rep", 3, 1, 2, 2048, 128, 128, 128, "bf16", "normalised", 5)
    host, dev = device_inputs(w)
    geo = so.geometry(w.T, w.chunk, w.d)
    cells, types = _assignment(w, geo, 1.0)
    prof, typ = torch.from_numpy(cells).cuda(), torch.from_numpy(types).cuda()
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype)
    first = plan.forward(dev["q"], dev["k"], dev["v"], prof=prof, type=typ).clone()
    for _ in range(20):
        assert torch.equal(plan.forward(dev["q"], dev["k"], dev["v"], prof=prof, type=typ), first)
    plan.check_status()
    lib = binding.load_library()
    ws = plan.workspace()
    args = [dev[x].data_ptr() for x in ("q", "k", "v")] + [first.data_ptr()]
    assert lib.smat_forward_routed(plan.handle, *args, None, typ.data_ptr(), ws.data_ptr(), ws.numel(), None) == 1
    assert lib.smat_forward_routed(plan.handle, *args, prof.data_ptr() + 2, typ.data_ptr(), ws.data_ptr(), ws.numel(), None) == 6
    with pytest.raises(ValueError):
        plan.forward(dev["q"], dev["k"], dev["v"], prof=prof[:, :-1].contiguous(), type=typ)
