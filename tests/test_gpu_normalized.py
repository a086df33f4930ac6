"""Normalised output on the GPU (smat_forward_normalized / smat_backward_normalized) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import smat_oracle as so
from paper_2609_36062_b200 import binding, synth
from tests.helpers import TOL, device_inputs, rel_err, sample_tokens, to_numpy64

pytestmark = pytest.mark.gpu

CASES = [
    # d, T, dk, dv, c, dtype, q
    (1, 256, 64, 64, 32, "f32", 0), (2, 512, 64, 64, 64, "f32", 0), (3, 512, 128, 64, 32, "f32", 0),
    (4, 1024, 64, 64, 16, "f32", 3), (3, 768, 64, 64, 64, "bf16", 0),
    (1, 1024, 128, 128, 128, "bf16", 0), (2, 1536, 128, 128, 64, "bf16", 0), (3, 2560, 128, 128, 128, "bf16", 0),
    (4, 2048, 128, 128, 128, "bf16", 0),
]


@pytest.mark.parametrize("d,T,dk,dv,c,dtype,q", CASES)
def test_normalised_forward_and_gradients_match_the_dense_oracle(d, T, dk, dv, c, dtype, q):
    w = synth.Workload("n", d, 1, 2, T, dk, dv, c, dtype, "positive", 41)
    host, dev = device_inputs(w, ("q", "k", "v", "do"))
    plan = binding.SmatPlan(1, 2, T, dk, dv, d, c, dtype, q_override=q, flags=binding.FLAG_NORMALIZED)
    O = plan.forward_normalized(dev["q"], dev["k"], dev["v"])
    dO = dev["do"].clone()
    dO[..., -1] = 0                                              # no upstream on the normaliser output
    dQ, dK, dV = plan.backward_normalized(dev["q"], dev["k"], dev["v"], O, dO)
    plan.check_status()
    M = so.dense_mask(T, c, d, q or None)
    tol = TOL[dtype]
    for h in range(w.bh):
        Q64, K64, V64, G64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v", "do"))
        ref, den = so.normalized_forward_dense(Q64, K64, V64[:, :-1], M)      # the library's value columns are 0 .. p-2
        got = to_numpy64(O[0, h])
        assert rel_err(got[:, :-1], ref) <= tol
        assert rel_err(got[:, -1], den) <= tol
        rq, rk, rv = so.normalized_backward_dense(Q64, K64, V64[:, :-1], G64[:, :-1], M)
        # dQ and dK are sums of a numerator part and a normaliser part that largely cancel (the output does not change
        # along the ray through Q).  Each part is an ordinary gradient of the linear pass and is held to the stated
        # tolerance at ITS scale; for fp32 inputs the sum itself meets the tolerance.
        dY = G64[:, :-1] / den[:, None]
        dz = -np.sum(G64[:, :-1] * ref, axis=1) / den
        Vbar = np.concatenate([V64[:, :-1], np.ones((T, 1))], axis=1)
        zero = np.zeros_like(dz)[:, None]
        num_part = so.backward_dense(Q64, K64, Vbar, np.concatenate([dY, zero], axis=1), M)
        den_part = so.backward_dense(Q64, K64, Vbar, np.concatenate([np.zeros_like(dY), dz[:, None]], axis=1), M)
        for idx, (name, g, r) in enumerate((("dQ", dQ, rq), ("dK", dK, rk))):
            err = float(np.max(np.abs(to_numpy64(g[0, h]) - r)))
            scale = float(np.max(np.abs(r))) if dtype == "f32" else max(float(np.max(np.abs(num_part[idx]))),
                                                                        float(np.max(np.abs(den_part[idx]))))
            assert err <= tol * scale, (name, h, err / scale)
        gv = to_numpy64(dV[0, h])
        assert rel_err(gv[:, :-1], rv) <= tol and not gv[:, -1].any()


def test_constant_values_come_back_unchanged_at_a_benchmark_shape():
    """Rows are convex combinations: V = const gives O = const whatever the mask and the features; sampled rows of a
    16 K-token problem against the oracle."""
    w = synth.Workload("n16", 4, 1, 2, 16384, 128, 128, 128, "bf16", "positive", 43)
    host, dev = device_inputs(w)
    plan = binding.SmatPlan(1, 2, w.T, 128, 128, 4, 128, "bf16", flags=binding.FLAG_NORMALIZED)
    assert plan.uses_tensor_cores()
    O = plan.forward_normalized(dev["q"], dev["k"], dev["v"])
    plan.check_status()
    geo = so.geometry(w.T, 128, 4)
    rows = sample_tokens(geo, 40, seed=1)
    Q64, K64, V64 = (synth.as_float64(w, host[x][1]) for x in ("q", "k", "v"))
    ref, den = so.normalized_forward_rows(Q64, K64, V64[:, :-1], geo, rows)
    got = to_numpy64(O[0, 1][rows])
    assert rel_err(got[:, :-1], ref) <= TOL["bf16"] and rel_err(got[:, -1], den) <= TOL["bf16"]
    const = torch.full_like(dev["v"], 1.5)
    Oc = plan.forward_normalized(dev["q"], dev["k"], const)
    assert float((Oc[..., :-1] - 1.5).abs().max()) <= 2e-2 * 1.5
    plain = binding.SmatPlan(1, 2, w.T, 128, 128, 4, 128, "bf16")
    with pytest.raises(binding.SmatError) as err:
        plain.forward_normalized(dev["q"], dev["k"], dev["v"])
    assert err.value.code == 10
