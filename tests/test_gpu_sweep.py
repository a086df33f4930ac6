"""GPU parity over a spread of geometries: every prime the tensor-core tabulation accepts (and two it does not),
both block shapes, several chunk widths — forward and gradients on sampled tokens against the fp64 oracle."""
import pytest

from oracle import smat_oracle as so
from paper_2609_36062_b200 import binding, synth
from tests.helpers import TOL, device_inputs, rel_err, sample_tokens, to_numpy64

pytestmark = pytest.mark.gpu

# d, T, chunk, q (0 = the default rule)
CASES = [
    (3, 1024, 128, 2), (3, 1536, 128, 3), (3, 2048, 64, 5), (3, 2304, 128, 7), (3, 2560, 128, 11), (3, 3072, 128, 19),
    (3, 2048, 128, 23),                     # q = 23: outside the resident-matrix kernel, bf16 tables summed on the ALUs
    (3, 2048, 128, 29), (3, 2560, 128, 31), # ... with the sums held in registers (K = 4 and K = 3 slopes per task)
    (3, 4096, 128, 37),                     # q = 37, the prime of the 64 K configuration with d = 3
    (3, 4096, 128, 41),                     # q = 41: no register-resident instance, sums straight from shared memory
    (4, 1024, 128, 2), (4, 1280, 128, 3), (4, 2048, 32, 13), (4, 1792, 128, 19), (4, 2048, 128, 0),
    (2, 1792, 128, 0), (2, 3072, 64, 29), (1, 1792, 128, 0),
]


@pytest.mark.parametrize("d,T,c,q", CASES)
def test_forward_and_gradients_on_sampled_tokens(d, T, c, q):
    w = synth.Workload("sweep", d, 1, 2, T, 128, 128, c, "bf16", "normalised", 100 + T // 128 + d)
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, q_override=q)
    assert plan.uses_tensor_cores()
    geo = so.geometry(T, c, d, q or None)
    O = plan.forward(dev["q"], dev["k"], dev["v"]).reshape(w.bh, T, -1)
    dQ, dK, dV = (g.reshape(w.bh, T, -1) for g in plan.backward(dev["q"], dev["k"], dev["v"], dev["do"]))
    plan.check_status()
    h = 1
    rows = sample_tokens(geo, 40, seed=7 + d)
    Q64, K64, V64, G64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v", "do"))
    assert rel_err(to_numpy64(O[h][rows]), so.forward_rows(Q64, K64, V64, geo, rows)) <= TOL["bf16"]
    rq = so.dq_rows(Q64, K64, V64, G64, geo, rows)
    rk, rv = so.dkdv_cols(Q64, K64, V64, G64, geo, rows)
    for name, g, r in (("dQ", dQ, rq), ("dK", dK, rk), ("dV", dV, rv)):
        e = rel_err(to_numpy64(g[h][rows]), r)
        assert e <= TOL["bf16"], (name, e)


def test_register_resident_and_shared_memory_tabulations_agree():
    """d = 3, q = 37: the register-resident sums (slab-major profile table) against the one-row-per-thread sums from
    shared memory (state-major table): same type table up to the order of the fp32 additions, same output."""
    import torch
    from paper_2609_36062_b200.binding import FLAG_D3_SHARED_SUMS
    w = synth.Workload("d3", 3, 1, 3, 4096, 128, 128, 128, "bf16", "normalised", 77)
    host, dev = device_inputs(w)
    outs, tables = [], []
    for flags in (0, FLAG_D3_SHARED_SUMS):
        plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, q_override=37, flags=flags)
        outs.append(plan.forward(dev["q"], dev["k"], dev["v"]))
        plan.check_status()
        F, U, _ = plan.debug_tables()
        tables.append((F, U))
    assert torch.equal(tables[0][0], tables[1][0])               # the pooled table is the same numbers in either layout
    assert rel_err(to_numpy64(tables[0][1]), to_numpy64(tables[1][1])) <= 8e-3
    assert rel_err(to_numpy64(outs[0]), to_numpy64(outs[1])) <= 1e-2
