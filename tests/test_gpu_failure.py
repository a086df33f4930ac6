"""The device-side failure path without a fault: a bounded wait that is meant to run out sets the status word, the
kernel returns normally, the host reads SMAT_ERR_DEVICE_TIMEOUT, and the context and the workspace stay usable."""
import numpy as np
import pytest
import torch

from oracle import smat_oracle as so
from paper_2609_36062_b200 import binding, synth
from tests.helpers import TOL, device_inputs, rel_err, to_numpy64

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_next_pass_is_clean():
    w = synth.Workload("probe", 3, 1, 2, 2048, 128, 128, 128, "bf16", "normalised", 17)
    host, dev = device_inputs(w)
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype)
    ws = plan.workspace()
    ref = plan.forward(dev["q"], dev["k"], dev["v"], workspace=ws).clone()
    plan.check_status(ws)                                        # clean after an ordinary pass
    binding.debug_timeout_probe(ws, limit_cycles=2_000_000)      # about a millisecond of SM clock, then it gives up
    with pytest.raises(binding.SmatError) as err:
        plan.check_status(ws)
    assert err.value.code == 9 and "wait" in binding.status_string(9)
    # the kernel returned normally: the context works, the next pass clears the word and reproduces the result
    out = plan.forward(dev["q"], dev["k"], dev["v"], workspace=ws)
    plan.check_status(ws)
    assert torch.equal(out, ref)
    geo = so.geometry(w.T, w.chunk, w.d)
    rows = [0, geo.n - 1, geo.n, geo.n + 5, w.T - 1]
    Q64, K64, V64 = (synth.as_float64(w, host[x][1]) for x in ("q", "k", "v"))
    assert rel_err(to_numpy64(out[0, 1][rows]), so.forward_rows(Q64, K64, V64, geo, rows)) <= TOL["bf16"]


def test_probe_rejects_bad_arguments():
    lib = binding.load_library()
    ws = torch.zeros(512, dtype=torch.uint8, device="cuda")
    assert lib.smat_debug_timeout_probe(None, 1000, None) == 1
    assert lib.smat_debug_timeout_probe(ws.data_ptr() + 8, 1000, None) == 6
    assert lib.smat_debug_timeout_probe(ws.data_ptr(), 0, None) == 2
    assert lib.smat_debug_timeout_probe(ws.data_ptr(), 1 << 40, None) == 2


def test_measured_add_rate_is_plausible():
    scalar = binding.measure_fadd_rate(packed=False)
    packed = binding.measure_fadd_rate(packed=True)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    nominal = sms * 128 * 1.965e9                                # lanes x maximum SM clock
    for rate in (scalar, packed):
        assert 0.3 * nominal <= rate <= 2.2 * nominal, (rate, nominal)
