"""Repeated launches: every device wait in the kernels is bounded and reports its expiry in the status word, so a
synchronisation race shows up as a rare expired wait (and a two-second launch) rather than as a wrong number.  A few
hundred back-to-back passes over shapes with many items per CTA must leave the status word clean and must reproduce
the first pass bit for bit."""
import pytest
import torch

from paper_2609_36062_b200 import binding, synth
from tests.helpers import device_inputs

pytestmark = pytest.mark.gpu

# d, batch, heads, T, d_v, chunk, passes: q = 13 with two CTAs per image and two issuing threads; q = 11 with both
# Radon stages in one launch; q = 17 with three slots per image
CASES = [(3, 4, 8, 4096, 128, 64, 300), (4, 1, 8, 16384, 128, 128, 100), (4, 1, 2, 65536, 128, 128, 40)]


@pytest.mark.parametrize("d,batch,heads,T,dv,c,passes", CASES)
def test_repeated_forward_passes_leave_the_status_clean(d, batch, heads, T, dv, c, passes):
    w = synth.Workload("soak", d, batch, heads, T, 128, dv, c, "bf16", "normalised", 300 + d)
    _, dev = device_inputs(w, ("q", "k", "v"))
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype)
    assert plan.uses_tensor_cores()
    first = plan.forward(dev["q"], dev["k"], dev["v"]).clone()
    plan.check_status()
    for i in range(passes):
        out = plan.forward(dev["q"], dev["k"], dev["v"])
        plan.check_status()          # the status word is cleared by the next pass: read it after each one
    assert torch.equal(out, first)


# d = 3 (q = 13, transposed Radon stage with three slots per image) and d = 4 (q = 11, both transposed stages in one launch)
@pytest.mark.parametrize("d,batch,heads,T,c,passes", [(3, 2, 8, 4096, 64, 100), (4, 1, 4, 16384, 128, 40)])
def test_repeated_backward_passes_leave_the_status_clean(d, batch, heads, T, c, passes):
    w = synth.Workload("soak", d, batch, heads, T, 128, 128, c, "bf16", "normalised", 311)
    _, dev = device_inputs(w, ("q", "k", "v", "do"))
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype)
    plan.forward(dev["q"], dev["k"], dev["v"])
    first = [g.clone() for g in plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])]
    plan.check_status()
    for i in range(passes):
        plan.forward(dev["q"], dev["k"], dev["v"])
        plan.check_status()
        grads = plan.backward(dev["q"], dev["k"], dev["v"], dev["do"])
        plan.check_status()
    for g, f in zip(grads, first):
        assert torch.equal(g, f)
