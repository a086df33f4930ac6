"""Scalar-gated SMat on the GPU (smat_forward_gated / smat_backward_gated) against the fp64 oracle of Eq. "gated"."""
import numpy as np
import pytest
import torch

from oracle import smat_oracle as so
from paper_2609_36062_b200 import binding, synth
from tests.helpers import TOL, device_inputs, rel_err, sample_tokens, to_numpy64

pytestmark = pytest.mark.gpu


def _gates(w, lo, seed):
    g = np.random.default_rng(seed)
    return np.log(g.uniform(lo, 1.0, (w.bh, w.T))).astype(np.float32)


CASES = [
    # d, T, dk, dv, c, dtype, q, smallest gate
    (1, 256, 64, 64, 32, "f32", 0, 0.8), (2, 512, 64, 64, 64, "f32", 0, 0.9), (3, 512, 128, 64, 32, "f32", 0, 0.7),
    (4, 1024, 64, 64, 16, "f32", 3, 0.9), (3, 768, 64, 64, 64, "bf16", 0, 0.9), (2, 384, 64, 128, 16, "f32", 0, 0.5),
    (3, 1024, 128, 128, 128, "bf16", 0, 0.95), (1, 512, 128, 128, 128, "bf16", 0, 0.9),
]


@pytest.mark.parametrize("d,T,dk,dv,c,dtype,q,lo", CASES)
def test_gated_forward_and_gradients_match_the_dense_oracle(d, T, dk, dv, c, dtype, q, lo):
    w = synth.Workload("g", d, 1, 2, T, dk, dv, c, dtype, "scaled", 21)
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    la = _gates(w, lo, 3)
    la_dev = torch.from_numpy(la).cuda()
    plan = binding.SmatPlan(1, 2, T, dk, dv, d, c, dtype, q_override=q, flags=binding.FLAG_GATED)
    assert not plan.uses_tensor_cores()
    # bf16 with 128-wide heads and blocks of whole 128-token tiles: the forward runs on the tensor-core kernels
    assert plan.gated_forward_uses_tensor_cores() == (dtype == "bf16" and dk == 128 and dv == 128 and (T // 2) % 128 == 0)
    O = plan.forward_gated(dev["q"], dev["k"], dev["v"], la_dev)
    dQ, dK, dV, dla = plan.backward_gated(dev["q"], dev["k"], dev["v"], la_dev, dev["do"])
    plan.check_status()
    M = so.dense_mask(T, c, d, q or None)
    tol = TOL[dtype]
    for h in range(w.bh):
        Q64, K64, V64, G64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v", "do"))
        lah = la[h].astype(np.float64)
        assert rel_err(to_numpy64(O[0, h]), so.gated_forward_dense(Q64, K64, V64, M, lah)) <= tol
        rq, rk, rv, rl = so.gated_backward_dense(Q64, K64, V64, G64, M, lah)
        for name, got, ref in (("dQ", dQ, rq), ("dK", dK, rk), ("dV", dV, rv)):
            e = rel_err(to_numpy64(got[0, h]), ref)
            assert e <= tol, (name, h, e)
        # the gate gradient is a difference of two row sums followed by a suffix sum over the whole sequence
        e = rel_err(dla[h].double().cpu().numpy(), rl)
        assert e <= (1e-3 if dtype == "f32" else 5e-2), ("dlog_a", h, e)


def test_unit_gates_reproduce_the_ungated_pass():
    w = synth.Workload("g1", 3, 1, 2, 512, 64, 64, 32, "f32", "scaled", 5)
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    zeros = torch.zeros(w.bh, w.T, device="cuda")
    gated = binding.SmatPlan(1, 2, w.T, 64, 64, 3, 32, "f32", flags=binding.FLAG_GATED)
    plain = binding.SmatPlan(1, 2, w.T, 64, 64, 3, 32, "f32")
    a = gated.forward_gated(dev["q"], dev["k"], dev["v"], zeros)
    b = plain.forward(dev["q"], dev["k"], dev["v"])
    assert rel_err(to_numpy64(a), to_numpy64(b)) <= 1e-6
    ga = gated.backward_gated(dev["q"], dev["k"], dev["v"], zeros, dev["do"])
    gb = plain.backward(dev["q"], dev["k"], dev["v"], dev["do"])
    for x, y in zip(ga[:3], gb):
        assert rel_err(to_numpy64(x), to_numpy64(y)) <= 1e-6


def test_strong_decay_stays_finite_and_matches_the_oracle():
    # λ reaches about -2000 at the end of the sequence: exp(-λ_j) alone would overflow fp32 after 13 tokens
    w = synth.Workload("g2", 3, 1, 1, 512, 64, 64, 32, "f32", "scaled", 6)
    host, dev = device_inputs(w)
    la = np.full((1, w.T), np.log(0.02), dtype=np.float32)
    plan = binding.SmatPlan(1, 1, w.T, 64, 64, 3, 32, "f32", flags=binding.FLAG_GATED)
    O = plan.forward_gated(dev["q"], dev["k"], dev["v"], torch.from_numpy(la).cuda())
    assert torch.isfinite(O).all()
    Q64, K64, V64 = (synth.as_float64(w, host[x][0]) for x in ("q", "k", "v"))
    ref = so.gated_forward_dense(Q64, K64, V64, so.dense_mask(w.T, 32, 3), la[0].astype(np.float64))
    assert rel_err(to_numpy64(O[0, 0]), ref) <= 1e-4


def test_gated_rows_at_a_longer_sequence_and_argument_errors():
    w = synth.Workload("g3", 3, 1, 2, 4096, 128, 128, 64, "bf16", "normalised", 9)
    host, dev = device_inputs(w)
    la = _gates(w, 0.97, 4)
    plan = binding.SmatPlan(1, 2, w.T, 128, 128, 3, 64, "bf16", flags=binding.FLAG_GATED)
    O = plan.forward_gated(dev["q"], dev["k"], dev["v"], torch.from_numpy(la).cuda())
    plan.check_status()
    geo = so.geometry(w.T, 64, 3)
    rows = sample_tokens(geo, 48, seed=2)
    Q64, K64, V64 = (synth.as_float64(w, host[x][1]) for x in ("q", "k", "v"))
    ref = so.gated_forward_rows(Q64, K64, V64, geo, la[1].astype(np.float64), rows)
    assert rel_err(to_numpy64(O[0, 1][rows]), ref) <= TOL["bf16"]
    # a plan without the flag has no room for λ and the rescaled copies
    plain = binding.SmatPlan(1, 2, w.T, 128, 128, 3, 64, "bf16")
    with pytest.raises(binding.SmatError) as err:
        plain.forward_gated(dev["q"], dev["k"], dev["v"], torch.from_numpy(la).cuda())
    assert err.value.code == 10


@pytest.mark.parametrize("d,T,c,q,lo", [(1, 2048, 128, 0, 0.97), (2, 4096, 128, 0, 0.95), (3, 4096, 64, 0, 0.9),
                                        (4, 2048, 128, 5, 0.98), (3, 8192, 128, 0, 0.999)])
def test_tensor_core_gated_forward_against_oracle_rows_and_the_alu_path(d, T, c, q, lo):
    w = synth.Workload("gtc", d, 1, 3, T, 128, 128, c, "bf16", "normalised", 31)
    host, dev = device_inputs(w)
    la = _gates(w, lo, 8)
    la_dev = torch.from_numpy(la).cuda()
    plan = binding.SmatPlan(1, 3, T, 128, 128, d, c, "bf16", q_override=q, flags=binding.FLAG_GATED)
    assert plan.gated_forward_uses_tensor_cores()
    O = plan.forward_gated(dev["q"], dev["k"], dev["v"], la_dev)
    plan.check_status()
    alu = binding.SmatPlan(1, 3, T, 128, 128, d, c, "bf16", q_override=q,
                           flags=binding.FLAG_GATED | binding.FLAG_SIMT_ONLY)
    assert not alu.gated_forward_uses_tensor_cores()
    O_alu = alu.forward_gated(dev["q"], dev["k"], dev["v"], la_dev)
    assert rel_err(to_numpy64(O), to_numpy64(O_alu)) <= 8e-3
    geo = so.geometry(T, c, d, q or None)
    rows = sample_tokens(geo, 64, seed=5)
    rows = np.unique(np.concatenate([rows, [0, 127, 128, geo.n - 1, geo.n, geo.n + 127, geo.n + 128, T - 1]]))
    for h in (0, 2):
        Q64, K64, V64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v"))
        ref = so.gated_forward_rows(Q64, K64, V64, geo, la[h].astype(np.float64), rows)
        assert rel_err(to_numpy64(O[0, h][rows]), ref) <= TOL["bf16"], (h,)
    # the pass is repeatable bit for bit
    O2 = plan.forward_gated(dev["q"], dev["k"], dev["v"], la_dev)
    assert torch.equal(O, O2)
    # gradients: the tensor-core backward against the fp32-ALU one (itself held to the dense oracle on small shapes)
    assert plan.gated_backward_uses_tensor_cores() and not alu.gated_backward_uses_tensor_cores()
    host2, dev2 = device_inputs(w, ("q", "k", "v", "do"))
    got = plan.backward_gated(dev2["q"], dev2["k"], dev2["v"], la_dev, dev2["do"])
    plan.check_status()
    ref = alu.backward_gated(dev2["q"], dev2["k"], dev2["v"], la_dev, dev2["do"])
    for name, x, y in zip(("dQ", "dK", "dV"), got[:3], ref[:3]):
        e = rel_err(to_numpy64(x), to_numpy64(y))
        assert e <= 8e-3, (name, e)
    e = rel_err(got[3].double().cpu().numpy(), ref[3].double().cpu().numpy())
    assert e <= 5e-2, ("dlog_a", e)
    if T <= 2048:   # and against the dense fp64 oracle where the T x T mask is small enough
        M = so.dense_mask(T, c, d, q or None)
        Q64, K64, V64, G64 = (synth.as_float64(w, host2[x][1]) for x in ("q", "k", "v", "do"))
        rq, rk, rv, rl = so.gated_backward_dense(Q64, K64, V64, G64, M, la[1].astype(np.float64))
        for name, x, r in (("dQ", got[0], rq), ("dK", got[1], rk), ("dV", got[2], rv)):
            assert rel_err(to_numpy64(x[0, 1]), r) <= TOL["bf16"], (name,)
        assert rel_err(got[3][1].double().cpu().numpy(), rl) <= 5e-2


def test_tensor_core_gated_forward_under_strong_decay():
    # λ falls by about 4 per token: exp(-λ_j) overflows after two dozen tokens; every exponent taken is a difference <= 0
    w = synth.Workload("gtc2", 3, 1, 2, 2048, 128, 128, 128, "bf16", "normalised", 32)
    host, dev = device_inputs(w)
    la = np.full((w.bh, w.T), np.log(0.02), dtype=np.float32)
    la[:, ::7] = np.log(0.9)
    plan = binding.SmatPlan(1, 2, w.T, 128, 128, 3, 128, "bf16", flags=binding.FLAG_GATED)
    assert plan.gated_forward_uses_tensor_cores()
    O = plan.forward_gated(dev["q"], dev["k"], dev["v"], torch.from_numpy(la).cuda())
    plan.check_status()
    assert torch.isfinite(O).all()
    geo = so.geometry(w.T, 128, 3)
    rows = sample_tokens(geo, 48, seed=6)
    Q64, K64, V64 = (synth.as_float64(w, host[x][1]) for x in ("q", "k", "v"))
    ref = so.gated_forward_rows(Q64, K64, V64, geo, la[1].astype(np.float64), rows)
    assert rel_err(to_numpy64(O[0, 1][rows]), ref) <= TOL["bf16"]


def test_unit_gates_on_the_tensor_core_path_reproduce_the_ungated_forward():
    w = synth.Workload("gtc3", 3, 1, 2, 4096, 128, 128, 128, "bf16", "normalised", 33)
    host, dev = device_inputs(w)
    zeros = torch.zeros(w.bh, w.T, device="cuda")
    gated = binding.SmatPlan(1, 2, w.T, 128, 128, 3, 128, "bf16", flags=binding.FLAG_GATED)
    plain = binding.SmatPlan(1, 2, w.T, 128, 128, 3, 128, "bf16", flags=binding.FLAG_PER_TILE_STATES)
    a = gated.forward_gated(dev["q"], dev["k"], dev["v"], zeros)
    b = plain.forward(dev["q"], dev["k"], dev["v"])
    # the gated tile adds its two accumulators in the epilogue: same sums, another order, so not the same bits
    assert rel_err(to_numpy64(a), to_numpy64(b)) <= 4e-3


def test_gated_backward_reuses_the_forward_tables_when_asked():
    w = synth.Workload("gkeep", 3, 1, 2, 4096, 128, 128, 128, "bf16", "normalised", 35)
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    la = torch.from_numpy(_gates(w, 0.95, 5)).cuda()
    keep = binding.SmatPlan(1, 2, w.T, 128, 128, 3, 128, "bf16", flags=binding.FLAG_GATED | binding.FLAG_KEEP_FORWARD_TABLES)
    full = binding.SmatPlan(1, 2, w.T, 128, 128, 3, 128, "bf16", flags=binding.FLAG_GATED)
    ws = keep.workspace(for_backward=True)
    keep.forward_gated(dev["q"], dev["k"], dev["v"], la, workspace=ws)
    a = keep.backward_gated(dev["q"], dev["k"], dev["v"], la, dev["do"], workspace=ws)
    n_kept = keep.last_launch_count()
    keep.check_status(ws)
    b = full.backward_gated(dev["q"], dev["k"], dev["v"], la, dev["do"])
    assert n_kept < full.last_launch_count()                 # no λ, no rescaled keys, no pooling, tabulation or state scan
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    # without a gated forward right before it, the same plan rebuilds everything
    c = keep.backward_gated(dev["q"], dev["k"], dev["v"], la, dev["do"], workspace=ws)
    assert keep.last_launch_count() == full.last_launch_count()
    for x, y in zip(c, b):
        assert torch.equal(x, y)


@pytest.mark.parametrize("flag", [binding.FLAG_ALU_TABULATION, binding.FLAG_ALG2_TABULATION])
def test_gated_passes_with_the_other_tabulations_of_the_inner_plan(flag):
    """The tabulation flags reach the plan that the gated passes run through: fp32 tables there send the typed read
    (and, for the literal Algorithm 2, the whole backward) to the fp32-ALU kernels; the results must not change."""
    w = synth.Workload("gflag", 3, 1, 2, 1024, 128, 128, 128, "bf16", "normalised", 36)
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    la = _gates(w, 0.93, 6)
    la_dev = torch.from_numpy(la).cuda()
    plan = binding.SmatPlan(1, 2, w.T, 128, 128, 3, 128, "bf16", flags=binding.FLAG_GATED | flag)
    assert plan.gated_forward_uses_tensor_cores()
    O = plan.forward_gated(dev["q"], dev["k"], dev["v"], la_dev)
    dQ, dK, dV, dla = plan.backward_gated(dev["q"], dev["k"], dev["v"], la_dev, dev["do"])
    plan.check_status()
    M = so.dense_mask(w.T, 128, 3)
    for h in range(w.bh):
        Q64, K64, V64, G64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v", "do"))
        lah = la[h].astype(np.float64)
        assert rel_err(to_numpy64(O[0, h]), so.gated_forward_dense(Q64, K64, V64, M, lah)) <= TOL["bf16"]
        rq, rk, rv, rl = so.gated_backward_dense(Q64, K64, V64, G64, M, lah)
        for name, got, ref in (("dQ", dQ, rq), ("dK", dK, rk), ("dV", dV, rv)):
            assert rel_err(to_numpy64(got[0, h]), ref) <= TOL["bf16"], (name, h)
        assert rel_err(dla[h].double().cpu().numpy(), rl) <= 5e-2
