"""CPU-side checks of the C boundary: the library loads, exports every declared symbol, validates its
arguments, and its integer routing matches the oracle bit for bit.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import smat_oracle as so
from paper_2609_36062_b200 import binding, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(smat_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    lib = binding.load_library()
    declared = _declared_symbols()
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), name
    assert set(binding.EXPORTS) <= declared


@pytest.mark.parametrize("name", list(synth.WORKLOADS))
def test_plan_geometry_matches_the_oracle(name):
    w = synth.WORKLOADS[name]
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype)
    g = plan.geometry()
    o = so.geometry(w.T, w.chunk, w.d)
    assert (g.n, g.m, g.q, g.P, g.A, g.B, g.nnzC) == (o.n, o.m, o.q, o.P, o.A, o.B, o.nnzC)
    assert g.vc_conditions_met == o.conditions_met
    assert plan.workspace_bytes(True) >= plan.workspace_bytes(False) > 0


@pytest.mark.parametrize("T,c,d,q", [(512, 64, 2, 0), (512, 64, 1, 0), (4096, 64, 3, 0), (2048, 32, 4, 0), (256, 16, 3, 5),
                                     (256, 16, 4, 3), (512, 16, 5, 3), (16384, 128, 4, 0), (8192, 64, 3, 0)])
def test_routing_indices_are_bit_exact(T, c, d, q):
    plan = binding.SmatPlan(1, 1, T, 64, 64, d, c, "f32", q_override=q)
    geo = so.geometry(T, c, d, q or None)
    prof, typ, ab = plan.routing_indices()
    o_prof, o_typ, o_ab = so.routing_tables(geo)
    assert np.array_equal(prof.numpy(), o_prof.reshape(prof.shape))
    assert np.array_equal(typ.numpy(), o_typ)
    assert np.array_equal(ab.numpy(), o_ab)


def test_argument_errors_are_reported_before_any_launch():
    lib = binding.load_library()
    h = ctypes.c_void_p()
    mk = lambda *a: lib.smat_plan_create(ctypes.byref(h), *a)
    assert lib.smat_plan_create(None, 1, 1, 512, 64, 64, 2, 64, 0, 0, 0) == 1          # null
    assert mk(1, 1, 512, 64, 64, 2, 64, 0, 7, 0) == 3                                   # dtype
    assert mk(1, 1, 512, 48, 64, 2, 64, 0, 0, 0) == 2                                   # d_k
    assert mk(1, 1, 500, 64, 64, 2, 64, 0, 0, 0) == 2                                   # T % chunk
    assert mk(1, 1, 512, 64, 64, 2, 48, 0, 0, 0) == 2                                   # chunk
    assert mk(1, 1, 512, 64, 64, 0, 64, 0, 0, 0) == 4                                   # d
    assert mk(1, 1, 512, 64, 64, 9, 64, 0, 0, 0) == 4
    assert mk(1, 1, 512, 64, 64, 2, 64, 15, 0, 0) == 4                                  # q not prime
    assert mk(1, 1, 64, 64, 64, 2, 64, 0, 0, 0) == 4                                    # T < 2c with d >= 2
    assert mk(1, 1, 64, 64, 64, 1, 64, 0, 0, 0) == 0                                    # ... but fine for d = 1
    plan = h.value
    # forward with null / short / misaligned buffers never launches
    assert lib.smat_forward(plan, None, 256, 256, 256, 256, 1 << 40, None) == 1
    assert lib.smat_forward(plan, 256, 256, 256, 256, None, 1 << 40, None) == 1
    assert lib.smat_forward(plan, 256, 256, 256, 256, 256, 16, None) == 5
    assert lib.smat_forward(plan, 256, 256, 256, 256, 264, 1 << 40, None) == 6
    assert lib.smat_forward(plan, 260, 256, 256, 256, 256, 1 << 40, None) == 6
    assert lib.smat_backward(plan, 256, 256, 256, None, 256, 256, 256, 256, 1 << 40, None) == 1
    assert lib.smat_workspace_bytes(None, 0) == 0
    lib.smat_plan_destroy(h)
    assert binding.status_string(5) == "workspace too small"


def test_binding_rejects_wrong_tensors():
    import torch
    plan = binding.SmatPlan(1, 1, 512, 64, 64, 2, 64, "f32")
    x = torch.zeros(1, 1, 512, 64)
    with pytest.raises(ValueError):
        plan.forward(x, x, x)          # CPU tensors: no fallback


def test_non_default_geometry_flags():
    g = binding.SmatPlan(1, 1, 256, 64, 64, 4, 16, "f32").geometry()   # default q too large for this T
    assert not g.vc_conditions_met
    g = binding.SmatPlan(1, 1, 256, 64, 64, 4, 16, "f32", q_override=2).geometry()
    assert g.vc_conditions_met and (g.P, g.B) == (8, 14)


def test_workspace_regions_follow_the_stored_element_types():
    """The bf16 tables and per-tile states of a tensor-core plan take half the bytes of their fp32 forms, and such a
    plan reserves no score-tile buffers; the plan is a function of the shape alone (no device is needed to size it)."""
    w = synth.WORKLOADS["t64k_d4"]
    plan = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype)
    assert plan.uses_tensor_cores() and plan.profile_table_element_bytes() == 2 and plan.type_table_element_bytes() == 2
    g = plan.geometry()
    state = w.d_k * w.d_v
    tables = w.bh * (g.P + g.B) * state * 2                      # F and U in bf16
    exchange = w.bh * (g.q ** 3 + g.q ** 2) * state * 2          # intermediate of the two d = 4 tabulation stages
    causal = w.bh * (w.T // 128) * state * 2
    rows = w.bh * w.T * 128 * 4                                  # long-range rows
    lists = w.bh * (w.T + g.P + g.B + 2) * 4                     # token lists of user-supplied routing (int32)
    need = tables + exchange + causal + rows + lists
    got = plan.workspace_bytes(False)
    assert need <= got <= need + 64 * 1024, (got, need)
    assert got < 9.0e9                                           # 15 GB with every region at 4 bytes per entry
    simt = binding.SmatPlan(w.batch, w.heads, w.T, w.d_k, w.d_v, w.d, w.chunk, w.dtype, flags=binding.FLAG_SIMT_ONLY)
    assert simt.workspace_bytes(False) > got
    # backward: adjoint tables in bf16 too, per-tile adjoint states
    back = plan.workspace_bytes(True)
    lr3 = w.bh * w.T * 128 * 2                                   # third buffer of bf16 long-range rows
    assert got + tables + causal + lr3 <= back <= got + tables + causal + lr3 + 64 * 1024


def test_launching_calls_report_a_missing_sm100_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present: the calls below would launch")
    lib = binding.load_library()
    h = ctypes.c_void_p()
    assert lib.smat_plan_create(ctypes.byref(h), 1, 1, 512, 64, 64, 2, 64, 0, 0, 0) == 0
    # all arguments are acceptable; what is missing is a compute capability 10.x device
    assert lib.smat_forward(h, 256, 256, 256, 256, 256, 1 << 40, None) == 7
    assert lib.smat_backward(h, 256, 256, 256, 256, 256, 256, 256, 256, 1 << 40, None) == 7
    assert lib.smat_forward_causal_static(256, 256, 256, 256, 1, 1, 128, None) == 7
    assert lib.smat_debug_timeout_probe(256, 1000, None) == 7
    assert "sm_100" in binding.status_string(7)
    lib.smat_plan_destroy(h)


@pytest.mark.parametrize("q", [2, 3, 5, 7, 11, 13, 17, 19, 23])
def test_tabulation_kernel_shared_memory_map_is_disjoint(q):
    """Ring slots, per-slot extra rows, the output-row table and the barrier words of the tensor-core tabulation kernel
    never overlap and no load box or staged tile leaves its slot, for every launch shape of every prime it accepts."""
    assert binding.load_library().smat_debug_tabulation_layout_ok(q) == 1


def test_gated_plans_size_their_inner_plan_and_decode_cache():
    """A gated plan on a tensor-core shape carries an ungated plan of its own for both passes: its workspace holds that
    plan's backward workspace as a region, its decode cache the bf16 type table, the running state and one word per
    head; other shapes, and SIMT_ONLY, have no inner plan and keep fp32 tables."""
    shape = (2, 4, 4096, 128, 128, 3, 64, "bf16")
    gated = binding.SmatPlan(*shape, flags=binding.FLAG_GATED)
    plain = binding.SmatPlan(*shape, flags=binding.FLAG_PER_TILE_STATES)
    alu = binding.SmatPlan(*shape, flags=binding.FLAG_GATED | binding.FLAG_SIMT_ONLY)
    assert not gated.uses_tensor_cores()                        # the gated plan itself keeps the fp32-ALU layout
    assert gated.gated_forward_uses_tensor_cores() and gated.gated_backward_uses_tensor_cores()
    assert not alu.gated_forward_uses_tensor_cores() and not alu.gated_backward_uses_tensor_cores()
    assert not plain.gated_forward_uses_tensor_cores()
    inner = plain.workspace_bytes(True)
    assert alu.workspace_bytes(False) + inner <= gated.workspace_bytes(False) <= alu.workspace_bytes(False) + inner + 4096
    assert gated.workspace_bytes(True) - gated.workspace_bytes(False) == alu.workspace_bytes(True) - alu.workspace_bytes(False)
    g = gated.geometry()
    bh, state = 8, 128 * 128
    lib = binding.load_library()
    assert lib.smat_decode_cache_bytes(gated.handle) == bh * g.B * state * 2 + bh * state * 4 + 256
    assert lib.smat_decode_cache_bytes(alu.handle) == bh * g.B * state * 4 + bh * state * 4 + 256
    assert lib.smat_decode_cache_bytes(plain.handle) == bh * g.B * state * 2 + bh * state * 4
    # the tabulation flags reach the inner plan: fp32 tables there (the literal Algorithm 2) mean an fp32-ALU gated backward
    odd = binding.SmatPlan(*shape, flags=binding.FLAG_GATED | binding.FLAG_ALG2_TABULATION)
    assert odd.gated_forward_uses_tensor_cores() and not odd.gated_backward_uses_tensor_cores()
    # a block boundary that is not a whole tile: no inner plan
    ragged = binding.SmatPlan(1, 2, 640, 128, 128, 3, 32, "bf16", flags=binding.FLAG_GATED)
    assert not ragged.gated_forward_uses_tensor_cores()
