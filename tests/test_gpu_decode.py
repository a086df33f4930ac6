"""GPU parity of cached decoding (Theorem "Streaming decoding") against the fp64 dense-mask oracle and the prefill."""
import numpy as np
import pytest
import torch

from oracle import chunkwise_ref as cw
from oracle import smat_oracle as so
from paper_2609_36062_b200 import binding, synth
from tests.helpers import TOL, device_inputs, rel_err, to_numpy64

pytestmark = pytest.mark.gpu

CASES = [
    (1, 512, 64, 64, 64, "f32", 0),
    (2, 512, 64, 64, 64, "f32", 0),
    (3, 1024, 64, 64, 32, "f32", 0),
    (4, 1024, 64, 64, 16, "f32", 3),
    (1, 1024, 128, 128, 128, "bf16", 0),      # one state: the sum over the whole distant block
    (2, 1024, 128, 128, 128, "bf16", 0),      # bf16 type table from the tensor-core pooling
    (3, 2048, 128, 128, 128, "bf16", 0),      # Radon stage on the tensor cores (d = 3)
    (4, 2048, 128, 128, 128, "bf16", 5),      # two Radon stages (d = 4)
    (3, 640, 128, 128, 32, "bf16", 0),        # n = 320 is not a multiple of 128: fp32-ALU tables for bf16 inputs
]


@pytest.mark.parametrize("d,T,dk,dv,c,dtype,q", CASES)
def test_decode_matches_dense_oracle_and_prefill(d, T, dk, dv, c, dtype, q):
    w = synth.Workload("dec", d, 1, 2, T, dk, dv, c, dtype, "scaled" if dtype == "f32" else "normalised", 13)
    host, dev = device_inputs(w)
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, q_override=q)
    geo = so.geometry(T, c, d, q or None)
    cache = plan.decode_cache()
    plan.decode_begin(dev["k"], dev["v"], cache)
    outs = []
    for t in range(geo.n, T):
        row = [dev[x][:, :, t].contiguous() for x in ("q", "k", "v")]
        outs.append(plan.decode_step(row[0], row[1], row[2], t, cache))
    plan.check_status()
    dec = torch.stack(outs, dim=2)                       # [batch, heads, m, d_v]
    prefill = plan.forward(dev["q"], dev["k"], dev["v"])
    plan.check_status()
    M = so.dense_mask(T, c, d, q or None)
    for h in range(w.bh):
        Q64, K64, V64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v"))
        ref = so.forward_dense(Q64, K64, V64, M)
        scale = np.abs(ref).max()
        got = to_numpy64(dec.reshape(w.bh, T - geo.n, dv)[h])
        assert np.abs(got - ref[geo.n:]).max() / scale <= TOL[dtype], (h, np.abs(got - ref[geo.n:]).max() / scale)
        pre = to_numpy64(prefill.reshape(w.bh, T, dv)[h][geo.n:])
        assert np.abs(got - pre).max() / scale <= (2e-5 if dtype == "f32" else 1.5e-2)
        if h == 0:   # and the streaming formula of the decoding proof, restated in fp64
            rows = list(range(geo.n, T, max(1, (T - geo.n) // 16)))
            stream = cw.streaming_rows(Q64, K64, V64, geo, rows)
            for t in rows:
                assert np.abs(got[t - geo.n] - stream[t]).max() / scale <= TOL[dtype]


def test_decode_rejects_tokens_outside_the_recent_block():
    w = synth.Workload("dec", 2, 1, 1, 512, 64, 64, 64, "f32", "scaled", 3)
    host, dev = device_inputs(w)
    plan = binding.SmatPlan(1, 1, 512, 64, 64, 2, 64, "f32")
    cache = plan.decode_cache()
    plan.decode_begin(dev["k"], dev["v"], cache)
    row = [dev[x][:, :, 0].contiguous() for x in ("q", "k", "v")]
    for t in (0, 255, 512):
        with pytest.raises(binding.SmatError):
            plan.decode_step(row[0], row[1], row[2], t, cache)
    with pytest.raises(binding.SmatError):
        plan.decode_step(row[0], row[1], row[2], 256, cache[:1024])


GATED_CASES = [
    (1, 512, 64, 64, 64, "f32", 0, 0.9), (2, 512, 64, 64, 64, "f32", 0, 0.8), (3, 1024, 64, 64, 32, "f32", 0, 0.95),
    (4, 1024, 64, 64, 16, "f32", 3, 0.9),
    (1, 1024, 128, 128, 128, "bf16", 0, 0.95), (3, 2048, 128, 128, 128, "bf16", 0, 0.97),   # tables by the tensor-core plan
    (4, 2048, 128, 128, 128, "bf16", 5, 0.98), (3, 640, 128, 128, 32, "bf16", 0, 0.9),      # n = 320: fp32-ALU tables
]


@pytest.mark.parametrize("d,T,dk,dv,c,dtype,q,lo", GATED_CASES)
def test_gated_decode_matches_dense_oracle_and_gated_prefill(d, T, dk, dv, c, dtype, q, lo):
    w = synth.Workload("gdec", d, 1, 2, T, dk, dv, c, dtype, "scaled" if dtype == "f32" else "normalised", 17)
    host, dev = device_inputs(w)
    la = np.log(np.random.default_rng(23).uniform(lo, 1.0, (w.bh, T))).astype(np.float32)
    la_dev = torch.from_numpy(la).cuda()
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, q_override=q,
                            flags=binding.FLAG_GATED)
    geo = so.geometry(T, c, d, q or None)
    cache = plan.decode_cache()
    plan.decode_begin_gated(dev["k"], dev["v"], la_dev, cache)
    outs = []
    for t in range(geo.n, T):
        row = [dev[x][:, :, t].contiguous() for x in ("q", "k", "v")]
        outs.append(plan.decode_step_gated(row[0], row[1], row[2], la_dev[:, t].contiguous(), t, cache))
    plan.check_status()
    dec = torch.stack(outs, dim=2)
    prefill = plan.forward_gated(dev["q"], dev["k"], dev["v"], la_dev)
    plan.check_status()
    M = so.dense_mask(T, c, d, q or None)
    for h in range(w.bh):
        Q64, K64, V64 = (synth.as_float64(w, host[x][h]) for x in ("q", "k", "v"))
        ref = so.gated_forward_dense(Q64, K64, V64, M, la[h].astype(np.float64))
        scale = np.abs(ref).max()
        got = to_numpy64(dec.reshape(w.bh, T - geo.n, dv)[h])
        assert np.abs(got - ref[geo.n:]).max() / scale <= TOL[dtype], (h, np.abs(got - ref[geo.n:]).max() / scale)
        pre = to_numpy64(prefill.reshape(w.bh, T, dv)[h][geo.n:])
        assert np.abs(got - pre).max() / scale <= (2e-5 if dtype == "f32" else 1.5e-2)
        if h == 1:   # the gated streaming recursion, restated in fp64
            rows = list(range(geo.n, T, max(1, (T - geo.n) // 16)))
            stream = cw.gated_streaming_rows(Q64, K64, V64, la[h].astype(np.float64), geo, rows)
            for t in rows:
                assert np.abs(got[t - geo.n] - stream[t]).max() / scale <= TOL[dtype]


def test_gated_and_plain_decode_calls_do_not_mix():
    w = synth.Workload("gdec2", 2, 1, 1, 512, 64, 64, 64, "f32", "scaled", 3)
    host, dev = device_inputs(w)
    la = torch.zeros(1, 512, device="cuda")
    gated = binding.SmatPlan(1, 1, 512, 64, 64, 2, 64, "f32", flags=binding.FLAG_GATED)
    plain = binding.SmatPlan(1, 1, 512, 64, 64, 2, 64, "f32")
    with pytest.raises(binding.SmatError) as err:
        gated.decode_begin(dev["k"], dev["v"], gated.decode_cache())
    assert err.value.code == 10
    with pytest.raises(binding.SmatError) as err:
        plain.decode_begin_gated(dev["k"], dev["v"], la, plain.decode_cache())
    assert err.value.code == 10
    # unit gates: the gated decoder reproduces the plain one
    cg, cp = gated.decode_cache(), plain.decode_cache()
    gated.decode_begin_gated(dev["k"], dev["v"], la, cg)
    plain.decode_begin(dev["k"], dev["v"], cp)
    for t in range(256, 272):
        row = [dev[x][:, :, t].contiguous() for x in ("q", "k", "v")]
        a = gated.decode_step_gated(row[0], row[1], row[2], la[:, t].contiguous(), t, cg)
        b = plain.decode_step(row[0], row[1], row[2], t, cp)
        assert rel_err(to_numpy64(a), to_numpy64(b)) <= 1e-6
