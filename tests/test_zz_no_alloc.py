"""The allocation-free causal forward (smat_forward_causal_static) against the fp64 oracle and against the
workspace-based smat_forward.

Runs last in the suite on purpose: if it fails, a run that stops at the first failure has already
exercised everything else.  It must also pass alone in a fresh process, where its first call is the one
that looks up the static scratch array."""
import pytest
import torch

from oracle import smat_oracle as so
from paper_2609_36062_b200 import binding, synth
from tests.helpers import TOL, device_inputs, rel_err, sample_tokens, to_numpy64

pytestmark = pytest.mark.gpu


def test_static_scratch_forward_matches_workspace_forward_twice_in_a_row():
    outs = []
    # two back-to-back calls with different inputs and shapes: the second one sees the first one's leftovers
    for seed, heads, T in ((41, 4, 2048), (42, 2, 1280)):
        w = synth.Workload("static", 1, 1, heads, T, 128, 128, 128, "bf16", "normalised", seed)
        host, dev = device_inputs(w)
        plan = binding.SmatPlan(w.batch, w.heads, w.T, 128, 128, 1, 128, "bf16")
        assert plan.uses_tensor_cores()
        ref = plan.forward(dev["q"], dev["k"], dev["v"])
        plan.check_status()
        out = torch.empty_like(ref)
        count = lambda: torch.cuda.memory_stats().get("allocation.all.allocated", 0)   # allocations made so far
        before = count()
        got = binding.forward_causal_static(dev["q"], dev["k"], dev["v"], out)
        assert count() == before                                 # nothing was allocated through torch either
        binding.static_check_status()                            # syncs; no bounded wait ran out on the static path
        assert count() == before
        err = rel_err(to_numpy64(got), to_numpy64(ref))
        assert err <= TOL["bf16"], err
        outs.append(err)
        # and against the oracle itself (d = 1: the causal mask), on sampled rows of the last head
        geo = so.geometry(T, 128, 1)
        rows = sample_tokens(geo, 48, seed=seed)
        Q64, K64, V64 = (synth.as_float64(w, host[x][heads - 1]) for x in ("q", "k", "v"))
        oracle_rows = so.forward_rows(Q64, K64, V64, geo, rows)
        assert rel_err(to_numpy64(got[0, heads - 1][rows]), oracle_rows) <= TOL["bf16"]
    assert max(outs) <= TOL["bf16"]


def test_static_scratch_rejects_problems_beyond_its_limit():
    lib = binding.load_library()
    tiles_over = binding.STATIC_MAX_TILES + 1
    x = torch.zeros(1, 1, 128, 128, dtype=torch.bfloat16, device="cuda")
    # shape arguments alone decide: no kernel is launched for an oversized request
    code = lib.smat_forward_causal_static(x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), 1, tiles_over, 128, None)
    assert code == 5 and "workspace" in binding.status_string(code)
    assert lib.smat_forward_causal_static(x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), 1, 1, 100, None) == 2
    assert lib.smat_forward_causal_static(None, x.data_ptr(), x.data_ptr(), x.data_ptr(), 1, 1, 128, None) == 1
