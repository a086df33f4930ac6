"""GPU parity: the CUDA path (through the C boundary) against the fp64 dense-mask oracle."""
import numpy as np
import pytest
import torch

from oracle import chunkwise_ref as cw
from oracle import smat_oracle as so
from paper_2609_36062_b200 import binding, synth
from tests.helpers import TOL, device_inputs, rel_err, sample_tokens, to_numpy64

pytestmark = pytest.mark.gpu


def _small(name, d, T, dk, dv, c, dtype, batch=1, heads=2, seed=11, recipe="scaled"):
    return synth.Workload(name, d, batch, heads, T, dk, dv, c, dtype, recipe, seed)


def _plan(w, q=0, flags=0):
    return binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, q_override=q, flags=flags)


# ---- routing: the mask as the device index code evaluates it ---------------------------------------
@pytest.mark.parametrize("T,c,d,q", [(512, 64, 1, 0), (512, 64, 2, 0), (1024, 32, 3, 0), (1024, 16, 4, 3),
                                     (512, 16, 5, 2), (4096, 64, 3, 0), (2048, 64, 4, 0)])
def test_device_mask_is_bit_exact(T, c, d, q):
    plan = binding.SmatPlan(1, 1, T, 64, 64, d, c, "f32", q_override=q)
    got = plan.debug_mask().cpu().numpy()
    ref = so.dense_mask(T, c, d, q or None)
    assert np.array_equal(got, ref)


# ---- full dense comparison on small shapes ---------------------------------------------------------
SMALL = [
    # d, T, dk, dv, c, dtype, q
    (1, 256, 64, 64, 32, "f32", 0),
    (2, 512, 64, 64, 64, "f32", 0),
    (2, 384, 64, 128, 16, "f32", 0),        # ragged: n = 192, mixed head dims
    (3, 512, 128, 64, 32, "f32", 0),
    (3, 768, 64, 64, 64, "bf16", 0),
    (4, 1024, 64, 64, 16, "f32", 3),
    (4, 512, 128, 128, 128, "bf16", 2),
    (5, 512, 64, 64, 16, "f32", 2),
    (3, 640, 128, 128, 128, "bf16", 0),     # T/c = 5: n = 256, m = 384
    (1, 1024, 128, 128, 128, "bf16", 0),    # tensor-core tiles, scan carried through the boundary
    (2, 1536, 128, 128, 64, "bf16", 0),     # caller's chunk 64 on 128-token tiles
    (3, 2560, 128, 128, 128, "bf16", 0),    # n = 1280: 10 tiles per block, longer than the TMEM ring
    (3, 320, 128, 128, 32, "bf16", 0),      # n = 160 is not a multiple of 128: fp32-ALU path for bf16 inputs
    (2, 8192, 128, 128, 128, "bf16", 0),    # q = 67: 61-62 tokens per profile, pooled on tensor cores, bf16 table
    (2, 2048, 128, 128, 128, "bf16", 2),    # two profiles of 512 tokens each: several 128-token passes per state
    (3, 4096, 128, 128, 64, "bf16", 0),     # q = 13: 12 tokens per profile on the tensor-core pooling path
]


@pytest.mark.parametrize("d,T,dk,dv,c,dtype,q", SMALL)
def test_forward_matches_dense_oracle(d, T, dk, dv, c, dtype, q):
    w = _small("s", d, T, dk, dv, c, dtype)
    host, dev = device_inputs(w)
    plan = _plan(w, q)
    O = plan.forward(dev["q"], dev["k"], dev["v"])
    plan.check_status()
    M = so.dense_mask(T, c, d, q or None)
    geo = so.geometry(T, c, d, q or None)
    F, U, Sin = plan.debug_tables()
    for h in range(w.bh):
        Q64, K64, V64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v"))
        ref = so.forward_dense(Q64, K64, V64, M)
        got = to_numpy64(O.reshape(w.bh, T, dv)[h])
        assert rel_err(got, ref) <= TOL[dtype], (h, rel_err(got, ref))
        if h == 0:   # intermediate tables against the chunkwise restatement (fp32 tables: tight bound)
            _, tab = cw.forward(Q64, K64, V64, geo, return_tables=True)
            if Sin is not None:
                ref_sin = tab["Sin"].copy()
                if d == 1:   # the library carries U_0 = F_0 across the boundary inside the scan
                    ref_sin[geo.n // c:] += tab["U"][0]
                    assert rel_err(to_numpy64(U[0]), tab["U"]) <= 1e-5
                assert rel_err(to_numpy64(Sin[0]), ref_sin) <= 1e-5
            if d > 1:
                # tensor-core plans with d >= 3 keep U in bf16 (it is only ever a bf16 MMA operand): one rounding
                # (bf16 profile table too where the tabulation runs on the tensor cores: up to three roundings in U)
                f_tol = 8e-3 if plan.profile_table_element_bytes() == 2 else 1e-5
                u_tol = (1.2e-2 if f_tol > 1e-5 and d > 2 else 8e-3) if plan.type_table_element_bytes() == 2 else 1e-5
                assert rel_err(to_numpy64(F[0]), tab["F"]) <= f_tol
                assert rel_err(to_numpy64(U[0]), tab["U"]) <= u_tol


@pytest.mark.parametrize("d,T,dk,dv,c,dtype,q", SMALL)
def test_backward_matches_dense_oracle(d, T, dk, dv, c, dtype, q):
    w = _small("s", d, T, dk, dv, c, dtype, seed=12)
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    plan = _plan(w, q)
    dQ, dK, dV = plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])
    plan.check_status()
    M = so.dense_mask(T, c, d, q or None)
    for h in range(w.bh):
        Q64, K64, V64, G64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v", "do"))
        rq, rk, rv = so.backward_dense(Q64, K64, V64, G64, M)
        for name, got, ref in (("dQ", dQ, rq), ("dK", dK, rk), ("dV", dV, rv)):
            g = to_numpy64(got.reshape(w.bh, T, -1)[h])
            assert rel_err(g, ref) <= TOL[dtype], (name, h, rel_err(g, ref))


@pytest.mark.parametrize("d,T,c,q", [(2, 512, 32, 0), (3, 1024, 32, 0), (3, 2048, 64, 13), (4, 1024, 16, 3), (4, 2048, 64, 5)])
@pytest.mark.parametrize("flags", [0, binding.FLAG_ALG2_TABULATION])
def test_tabulation_variants_match_algorithm2(d, T, c, q, flags):
    """Both the staged sums and the direct double loop of Algorithm 2 must give the oracle's type table,
    and the transposed tabulation of the backward pass its adjoint."""
    w = _small("tab", d, T, 64, 64, c, "f32", heads=1, seed=21)
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    plan = _plan(w, q, flags)
    geo = so.geometry(T, c, d, q or None)
    plan.forward(dev["q"], dev["k"], dev["v"])
    F, U, _ = plan.debug_tables()
    Q64, K64, V64, G64 = (synth.as_float64(w, host[x][0]) for x in ("q", "k", "v", "do"))
    _, tab = cw.forward(Q64, K64, V64, geo, return_tables=True)
    assert rel_err(to_numpy64(F[0]), tab["F"]) <= 1e-5
    assert rel_err(to_numpy64(U[0]), tab["U"]) <= 1e-5
    dQ, dK, dV = plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])
    M = so.dense_mask(T, c, d, q or None)
    for got, ref in zip((dQ, dK, dV), so.backward_dense(Q64, K64, V64, G64, M)):
        assert rel_err(to_numpy64(got[0, 0]), ref) <= 1e-4


@pytest.mark.parametrize("d,T,q", [(3, 2048, 5), (3, 4096, 13), (3, 4096, 17), (3, 4096, 19), (4, 2048, 5), (4, 4096, 7),
                                   (4, 4096, 11), (4, 4096, 17)])
def test_tensor_core_tabulation_matches_the_incidence_sums(d, T, q):
    """Radon stages on the tensor cores (bf16 tables): F against the pooled outer products, sampled rows of U against
    U_h = sum of F_x over the points of hyperplane h (Algorithm 2) written out with the oracle's incidence matrix, the
    output against the fp32-ALU tabulation, and the gradients (transposed stages) against that path too."""
    w = _small("tabtc", d, T, 128, 128, 128, "bf16", heads=1, seed=81, recipe="normalised")
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    tc_plan, alu_plan = _plan(w, q), _plan(w, q, flags=binding.FLAG_ALU_TABULATION)
    assert tc_plan.type_table_element_bytes() == 2
    out_tc = tc_plan.forward(dev["q"], dev["k"], dev["v"])
    tc_plan.check_status()
    F, U, _ = tc_plan.debug_tables()
    geo = so.geometry(T, 128, d, q)
    K64, V64 = (synth.as_float64(w, host[x][0]) for x in ("k", "v"))
    Fref = np.zeros((geo.P, 128, 128))
    for t in range(geo.n):
        Fref[t % geo.P] += np.outer(K64[t], V64[t])
    F64 = to_numpy64(F[0])
    assert rel_err(F64, Fref) <= 4e-3          # one bf16 rounding of each entry
    pts = [so.prof(v, geo) for v in range(geo.P)]
    rng = np.random.default_rng(5)
    types = np.unique(np.concatenate([[0, q - 1, q, geo.B - q - 1, geo.B - q, geo.B - 1], rng.integers(0, geo.B, 24)]))
    U64 = to_numpy64(U[0][torch.as_tensor(types, device=U.device)])
    for i, h in enumerate(types):
        a, b = so.type_pair(int(h), geo)
        ref = Fref[[v for v, x in enumerate(pts) if so.on_hyperplane(x, a, b, geo.q)]].sum(axis=0)
        scale = max(np.abs(ref).max(), 1e-30)
        assert np.abs(U64[i] - ref).max() / scale <= 1.5e-2, (h, np.abs(U64[i] - ref).max() / scale)
    out_alu = alu_plan.forward(dev["q"], dev["k"], dev["v"])
    alu_plan.check_status()
    assert rel_err(to_numpy64(out_tc), to_numpy64(out_alu)) <= 1e-2
    g_tc = tc_plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])
    tc_plan.check_status()
    g_alu = alu_plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])
    for name, a, b in zip(("dQ", "dK", "dV"), g_tc, g_alu):
        assert rel_err(to_numpy64(a), to_numpy64(b)) <= 2e-2, name


def test_tensor_core_and_alu_paths_agree():
    """The same bf16 problem through the tcgen05 kernels and through the fp32-ALU kernels."""
    w = _small("tc", 3, 2048, 128, 128, 128, "bf16", heads=2, seed=31, recipe="normalised")
    host, dev = device_inputs(w)
    tc_plan, alu_plan = _plan(w), _plan(w, flags=binding.FLAG_SIMT_ONLY)
    assert tc_plan.uses_tensor_cores() and not alu_plan.uses_tensor_cores()
    a = to_numpy64(tc_plan.forward(dev["q"], dev["k"], dev["v"]))
    tc_plan.check_status()
    b = to_numpy64(alu_plan.forward(dev["q"], dev["k"], dev["v"]))
    assert rel_err(a, b) <= 1e-2


@pytest.mark.parametrize("d,T,q", [(1, 4096, 0), (3, 4096, 0), (2, 2560, 0), (4, 8192, 0)])
def test_two_level_and_per_tile_causal_branches_agree(d, T, q):
    """Segment form (one fp32 state per segment of tiles) against the per-tile form, and both against the oracle."""
    w = _small("seg", d, T, 128, 128, 128, "bf16", heads=3, seed=51, recipe="normalised")
    host, dev = device_inputs(w)
    seg_plan, tile_plan = _plan(w, q), _plan(w, q, flags=binding.FLAG_PER_TILE_STATES)
    a = seg_plan.forward(dev["q"], dev["k"], dev["v"])
    seg_plan.check_status()
    b = tile_plan.forward(dev["q"], dev["k"], dev["v"])
    tile_plan.check_status()
    geo = so.geometry(T, 128, d, q or None)
    rows = sample_tokens(geo, 64, seed=3)
    Q64, K64, V64 = (synth.as_float64(w, host[x][1]) for x in ("q", "k", "v"))
    ref = so.forward_rows(Q64, K64, V64, geo, rows)
    for out in (a, b):
        assert rel_err(to_numpy64(out[0, 1][rows]), ref) <= TOL["bf16"]
    assert rel_err(to_numpy64(a), to_numpy64(b)) <= 1e-2


@pytest.mark.parametrize("d,T,q", [(1, 2048, 0), (2, 4096, 0), (3, 4096, 0), (3, 2560, 0), (4, 4096, 0), (2, 1024, 0)])
def test_tensor_core_backward_matches_oracle_and_alu_path(d, T, q):
    """smat_backward on the tcgen05 path against sampled oracle gradients and against the fp32-ALU path."""
    w = _small("tcb", d, T, 128, 128, 128, "bf16", heads=2, seed=61, recipe="normalised")
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    tc_plan, alu_plan = _plan(w, q), _plan(w, q, flags=binding.FLAG_SIMT_ONLY)
    assert tc_plan.uses_tensor_cores()
    got = tc_plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])
    tc_plan.check_status()
    ref_alu = alu_plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])
    geo = so.geometry(T, 128, d, q or None)
    rows = sample_tokens(geo, 48, seed=9)
    Q64, K64, V64, G64 = (synth.as_float64(w, host[x][1]) for x in ("q", "k", "v", "do"))
    rq = so.dq_rows(Q64, K64, V64, G64, geo, rows)
    rk, rv = so.dkdv_cols(Q64, K64, V64, G64, geo, rows)
    for name, g, a, r in (("dQ", got[0], ref_alu[0], rq), ("dK", got[1], ref_alu[1], rk), ("dV", got[2], ref_alu[2], rv)):
        e = rel_err(to_numpy64(g[0, 1][rows]), r)
        assert e <= TOL["bf16"], (name, e)
        assert rel_err(to_numpy64(g), to_numpy64(a)) <= 2e-2, name


def test_backward_with_kept_forward_tables_matches_rebuilding_them():
    w = _small("keep", 3, 4096, 128, 128, 128, "bf16", heads=2, seed=71, recipe="normalised")
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    keep, rebuild = _plan(w, flags=binding.FLAG_KEEP_FORWARD_TABLES), _plan(w)
    ws = keep.workspace(for_backward=True)
    keep.forward(dev["q"], dev["k"], dev["v"], workspace=ws)
    a = keep.backward(dev["q"], dev["k"], dev["v"], dev["do"], workspace=ws)
    keep.check_status(ws)
    b = rebuild.backward(dev["q"], dev["k"], dev["v"], dev["do"])
    assert keep.last_launch_count() < rebuild.last_launch_count()
    # The kept pass takes the per-tile incoming states the forward's segment kernel published (segment state + the
    # tiles of the segment, summed in tensor memory) instead of re-scanning K, V tile by tile: the same fp32 sums in a
    # different order, rounded to bf16 once either way.
    for x, y in zip(a, b):
        assert rel_err(to_numpy64(x), to_numpy64(y)) <= 4e-3
    geo = so.geometry(w.T, w.chunk, w.d)
    rows = sample_tokens(geo, 40, seed=4)
    Q64, K64, V64, G64 = (synth.as_float64(w, host[x][1]) for x in ("q", "k", "v", "do"))
    rq = so.dq_rows(Q64, K64, V64, G64, geo, rows)
    rk, rv = so.dkdv_cols(Q64, K64, V64, G64, geo, rows)
    for g, r in zip(a, (rq, rk, rv)):
        assert rel_err(to_numpy64(g[0, 1][rows]), r) <= TOL["bf16"]


def test_chunk_size_invariance_on_device():
    outs = []
    for c in (16, 32, 64, 128):
        w = _small("inv", 2, 512, 64, 64, c, "f32", seed=5)
        host, dev = device_inputs(w)
        outs.append(to_numpy64(_plan(w).forward(dev["q"], dev["k"], dev["v"])))
    for o in outs[1:]:
        assert rel_err(o, outs[0]) <= 2e-6


def test_degenerate_shapes():
    # T = 2c (one chunk per block), a single chunk with d = 1, and P > n (empty profile cells)
    for (d, T, c, q) in [(2, 128, 64, 0), (1, 64, 64, 0), (3, 64, 16, 7)]:
        w = _small("deg", d, T, 64, 64, c, "f32", heads=1)
        host, dev = device_inputs(w, ("q", "k", "v", "do"))
        plan = _plan(w, q)
        O = plan.forward(dev["q"], dev["k"], dev["v"])
        dQ, dK, dV = plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])
        M = so.dense_mask(T, c, d, q or None)
        Q64, K64, V64, G64 = (synth.as_float64(w, host[x][0]) for x in ("q", "k", "v", "do"))
        assert rel_err(to_numpy64(O[0, 0]), so.forward_dense(Q64, K64, V64, M)) <= 1e-4
        for got, ref in zip((dQ, dK, dV), so.backward_dense(Q64, K64, V64, G64, M)):
            assert rel_err(to_numpy64(got[0, 0]), ref) <= 1e-4


# ---- the benchmark configurations --------------------------------------------------------------------
def test_config1_full_dense():
    for name in ("small_d2", "small_d1"):
        w = synth.WORKLOADS[name]
        host, dev = device_inputs(w, ("q", "k", "v", "do"))
        plan = _plan(w)
        O = plan.forward(dev["q"], dev["k"], dev["v"])
        dQ, dK, dV = plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])
        plan.check_status()
        M = so.dense_mask(w.T, w.chunk, w.d)
        Q64, K64, V64, G64 = (synth.as_float64(w, host[x][0]) for x in ("q", "k", "v", "do"))
        assert rel_err(to_numpy64(O[0, 0]), so.forward_dense(Q64, K64, V64, M)) <= 1e-4
        for got, ref in zip((dQ, dK, dV), so.backward_dense(Q64, K64, V64, G64, M)):
            assert rel_err(to_numpy64(got[0, 0]), ref) <= 1e-4


def _check_sampled(w, heads_to_check, nrows, backward=False, dense_head=None):
    tensors = ("q", "k", "v", "do") if backward else ("q", "k", "v")
    host, dev = device_inputs(w, tensors)
    plan = _plan(w)
    geo = so.geometry(w.T, w.chunk, w.d)
    O = plan.forward(dev["q"], dev["k"], dev["v"])
    grads = plan.backward(dev["q"], dev["k"], dev["v"], dev["do"]) if backward else None
    plan.check_status()
    O = O.reshape(w.bh, w.T, w.d_v)
    tol = TOL[w.dtype]
    for h in heads_to_check:
        Q64, K64, V64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v"))
        rows = sample_tokens(geo, nrows, seed=100 + h)
        ref = so.forward_rows(Q64, K64, V64, geo, rows)
        got = to_numpy64(O[h][rows])
        # normalise by the largest entry of the whole output, which the sampled rows at the end reach
        assert rel_err(got, ref) <= tol, ("O", h, rel_err(got, ref))
        if backward:
            G64 = synth.as_float64(w, host["do"][h])
            dQ, dK, dV = (g.reshape(w.bh, w.T, -1)[h] for g in grads)
            rq = so.dq_rows(Q64, K64, V64, G64, geo, rows)
            rk, rv = so.dkdv_cols(Q64, K64, V64, G64, geo, rows)
            for name, g, r in (("dQ", dQ, rq), ("dK", dK, rk), ("dV", dV, rv)):
                e = rel_err(to_numpy64(g[rows]), r)
                assert e <= tol, (name, h, e)
    if dense_head is not None:
        h = dense_head
        Q64, K64, V64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v"))
        ref = so.forward_dense(Q64, K64, V64, so.dense_mask(w.T, w.chunk, w.d))
        assert rel_err(to_numpy64(O[h]), ref) <= tol


def test_config2_t4k_d3():
    w = synth.WORKLOADS["t4k_d3"]
    _check_sampled(w, heads_to_check=[0, 13, w.bh - 1], nrows=96, dense_head=5)


def test_config3_t16k_d4():
    w = synth.WORKLOADS["t16k_d4"]
    _check_sampled(w, heads_to_check=[0, 17, w.bh - 1], nrows=96)


@pytest.mark.parametrize("name", ["t64k_d1", "t64k_d2", "t64k_d3", "t64k_d4"])
def test_config4_t64k(name):
    w = synth.WORKLOADS[name]
    _check_sampled(w, heads_to_check=[0, w.bh - 1], nrows=64)


def test_config5_t8k_d3_forward_backward():
    w = synth.WORKLOADS["t8k_d3_fwdbwd"]
    _check_sampled(w, heads_to_check=[0, 77, w.bh - 1], nrows=64, backward=True)


@pytest.mark.parametrize("d,T", [(1, 2048), (2, 4096), (3, 4096), (4, 4096)])
def test_fused_and_separate_tile_adjoints_agree(d, T):
    """The one-kernel form of the three within-chunk adjoints against three launches of the general tile kernel."""
    w = _small("fused", d, T, 128, 128, 128, "bf16", heads=3, seed=91, recipe="normalised")
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    fused, separate = _plan(w), _plan(w, flags=binding.FLAG_SEPARATE_TILE_ADJOINTS)
    a = fused.backward(dev["q"], dev["k"], dev["v"], dev["do"])
    fused.check_status()
    b = separate.backward(dev["q"], dev["k"], dev["v"], dev["do"])
    separate.check_status()
    # one tile kernel instead of three, and (d >= 2) one read of the per-profile adjoint states instead of two
    assert fused.last_launch_count() == separate.last_launch_count() - (2 if d == 1 else 3)
    for x, y in zip(a, b):
        assert rel_err(to_numpy64(x), to_numpy64(y)) <= 2e-3


# ---- the "next" rows at the sizes and in the launch configuration bench.py times ---------------------------------
def _bench_plan(w):
    flags = {"gated": binding.FLAG_GATED, "normalized": binding.FLAG_NORMALIZED}.get(w.variant, 0)
    return binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, flags=flags)


def test_bench_workload_hashed_routing_sampled_rows():
    w = synth.WORKLOADS["t16k_d4_hashed"]
    host, dev = device_inputs(w)
    plan = _bench_plan(w)
    geo = so.geometry(w.T, w.chunk, w.d)
    prof = np.stack([synth.hashed_cells(w, h, geo.n, geo.P) for h in range(w.bh)])
    typ = np.stack([synth.hashed_types(w, h, geo.m, geo.B) for h in range(w.bh)])
    O = plan.forward(dev["q"], dev["k"], dev["v"], prof=torch.from_numpy(prof).cuda(), type=torch.from_numpy(typ).cuda())
    plan.check_status()
    O = O.reshape(w.bh, w.T, w.d_v)
    for h in (0, w.bh - 1):
        Q64, K64, V64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v"))
        rows = sample_tokens(geo, 64, seed=300 + h)
        ref = so.routed_forward_rows(Q64, K64, V64, geo, prof[h], typ[h], rows)
        assert rel_err(to_numpy64(O[h][rows]), ref) <= TOL[w.dtype], (h,)


def test_bench_workload_normalized_sampled_rows():
    w = synth.WORKLOADS["t16k_d4_normalized"]
    host, dev = device_inputs(w)
    plan = _bench_plan(w)
    geo = so.geometry(w.T, w.chunk, w.d)
    O = plan.forward_normalized(dev["q"], dev["k"], dev["v"])
    plan.check_status()
    O = O.reshape(w.bh, w.T, w.d_v)
    for h in (0, w.bh - 1):
        Q64, K64, V64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v"))
        rows = sample_tokens(geo, 64, seed=400 + h)
        ref, den = so.normalized_forward_rows(Q64, K64, V64[:, :-1], geo, rows)
        got = to_numpy64(O[h][rows])
        assert rel_err(got[:, :-1], ref) <= TOL[w.dtype], (h,)
        assert rel_err(got[:, -1], den) <= TOL[w.dtype], (h,)            # the last column carries the normaliser


@pytest.mark.parametrize("name", ["t4k_d3_gated", "t4k_d3_gated_fwdbwd"])
def test_bench_workload_gated(name):
    w = synth.WORKLOADS[name]
    tensors = ("q", "k", "v", "do") if w.backward else ("q", "k", "v")
    host, dev = device_inputs(w, tensors)
    plan = _bench_plan(w)
    assert plan.gated_forward_uses_tensor_cores()
    geo = so.geometry(w.T, w.chunk, w.d)
    la = np.stack([synth.log_gates(w, h) for h in range(w.bh)])
    la_dev = torch.from_numpy(la).cuda()
    O = plan.forward_gated(dev["q"], dev["k"], dev["v"], la_dev)
    grads = plan.backward_gated(dev["q"], dev["k"], dev["v"], la_dev, dev["do"]) if w.backward else None
    plan.check_status()
    O = O.reshape(w.bh, w.T, w.d_v)
    for h in (0, w.bh - 1):
        Q64, K64, V64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v"))
        rows = sample_tokens(geo, 64, seed=500 + h)
        ref = so.gated_forward_rows(Q64, K64, V64, geo, la[h].astype(np.float64), rows)
        assert rel_err(to_numpy64(O[h][rows]), ref) <= TOL[w.dtype], (h,)
    if w.backward:   # one head against the dense fp64 adjoint (T = 4096: the mask is 16 M entries)
        h = w.bh - 1
        Q64, K64, V64, G64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v", "do"))
        M = so.dense_mask(w.T, w.chunk, w.d)
        rq, rk, rv, rl = so.gated_backward_dense(Q64, K64, V64, G64, M, la[h].astype(np.float64))
        dQ, dK, dV = (g.reshape(w.bh, w.T, -1)[h] for g in grads[:3])
        for nm, g, r in (("dQ", dQ, rq), ("dK", dK, rk), ("dV", dV, rv)):
            assert rel_err(to_numpy64(g), r) <= TOL[w.dtype], (nm,)
        assert rel_err(grads[3].reshape(w.bh, w.T)[h].double().cpu().numpy(), rl) <= 5e-2
