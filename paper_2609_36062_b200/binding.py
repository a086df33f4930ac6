"""Thin ctypes binding of libsmat.so: argument marshalling only, same names as the C boundary.

Every step of the path runs inside the library's CUDA kernels.  PyTorch is used for device
memory and streams.  There is no CPU fallback: if the shared library is missing or the device
is absent the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsmat.so")

SMAT_F32, SMAT_BF16 = 0, 1
FLAG_SIMT_ONLY = 1
FLAG_ALG2_TABULATION = 2
FLAG_PER_TILE_STATES = 4
FLAG_KEEP_FORWARD_TABLES = 8
FLAG_ALU_TABULATION = 16
FLAG_D3_SHARED_SUMS = 32
FLAG_GATED = 64
FLAG_NORMALIZED = 128
FLAG_SEPARATE_TILE_ADJOINTS = 256

EXPORTS = [
    "smat_plan_create", "smat_plan_destroy", "smat_get_geometry", "smat_workspace_bytes", "smat_forward",
    "smat_backward", "smat_routing_indices", "smat_debug_mask", "smat_debug_tables", "smat_check_status",
    "smat_last_launch_count", "smat_status_string", "smat_profile_enable", "smat_profile_read", "smat_uses_tensor_cores", "smat_gated_forward_uses_tensor_cores", "smat_gated_backward_uses_tensor_cores", "smat_forward_causal_static", "smat_type_table_element_bytes",
    "smat_profile_table_element_bytes", "smat_decode_cache_bytes", "smat_decode_begin", "smat_decode_step", "smat_decode_begin_gated", "smat_decode_step_gated",
    "smat_static_check_status", "smat_debug_timeout_probe", "smat_measure_fadd_rate",
    "smat_forward_routed", "smat_backward_routed", "smat_forward_gated", "smat_backward_gated",
    "smat_forward_normalized", "smat_backward_normalized", "smat_debug_tabulation_layout_ok",
]


class SmatError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: status {code} ({status_string(code)})")
        self.code = code


class _Geometry(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int64), ("c", ctypes.c_int64), ("n", ctypes.c_int64), ("m", ctypes.c_int64),
                ("d", ctypes.c_int32), ("q", ctypes.c_int32), ("P", ctypes.c_int64), ("A", ctypes.c_int64),
                ("B", ctypes.c_int64), ("nnzC", ctypes.c_int64), ("vc_conditions_met", ctypes.c_int32)]


@dataclass(frozen=True)
class Geometry:
    T: int
    c: int
    n: int
    m: int
    d: int
    q: int
    P: int
    A: int
    B: int
    nnzC: int
    vc_conditions_met: bool


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libsmat.so (built in-tree by paper_2609_36062_b200.build); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} not found: build it with `python -m paper_2609_36062_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
    lib.smat_plan_create.argtypes = [ctypes.POINTER(vp), i, i, i64, i, i, i, i, i, i, ctypes.c_uint]
    lib.smat_plan_create.restype = i
    lib.smat_plan_destroy.argtypes = [vp]
    lib.smat_plan_destroy.restype = None
    lib.smat_get_geometry.argtypes = [vp, ctypes.POINTER(_Geometry)]
    lib.smat_get_geometry.restype = i
    lib.smat_workspace_bytes.argtypes = [vp, i]
    lib.smat_workspace_bytes.restype = sz
    lib.smat_forward.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    lib.smat_forward.restype = i
    lib.smat_backward.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.smat_backward.restype = i
    lib.smat_forward_routed.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.smat_forward_routed.restype = i
    lib.smat_backward_routed.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.smat_backward_routed.restype = i
    lib.smat_forward_gated.argtypes = [vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.smat_forward_gated.restype = i
    lib.smat_backward_gated.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.smat_backward_gated.restype = i
    lib.smat_forward_normalized.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    lib.smat_forward_normalized.restype = i
    lib.smat_backward_normalized.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.smat_backward_normalized.restype = i
    lib.smat_debug_tabulation_layout_ok.argtypes = [i]
    lib.smat_debug_tabulation_layout_ok.restype = i
    lib.smat_routing_indices.argtypes = [vp, vp, vp, vp]
    lib.smat_routing_indices.restype = i
    lib.smat_debug_mask.argtypes = [vp, vp, vp]
    lib.smat_debug_mask.restype = i
    lib.smat_debug_tables.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.smat_debug_tables.restype = i
    lib.smat_check_status.argtypes = [vp, vp, vp]
    lib.smat_check_status.restype = i
    lib.smat_last_launch_count.argtypes = [vp]
    lib.smat_last_launch_count.restype = i
    lib.smat_type_table_element_bytes.argtypes = [vp]
    lib.smat_type_table_element_bytes.restype = i
    lib.smat_decode_cache_bytes.argtypes = [vp]
    lib.smat_decode_cache_bytes.restype = ctypes.c_size_t
    lib.smat_decode_begin.argtypes = [vp, vp, vp, vp, ctypes.c_size_t, vp, ctypes.c_size_t, vp]
    lib.smat_decode_begin.restype = i
    lib.smat_decode_step.argtypes = [vp, vp, vp, vp, i64, vp, vp, ctypes.c_size_t, vp]
    lib.smat_decode_step.restype = i
    lib.smat_decode_begin_gated.argtypes = [vp, vp, vp, vp, vp, ctypes.c_size_t, vp, ctypes.c_size_t, vp]
    lib.smat_decode_begin_gated.restype = i
    lib.smat_decode_step_gated.argtypes = [vp, vp, vp, vp, vp, i64, vp, vp, ctypes.c_size_t, vp]
    lib.smat_decode_step_gated.restype = i
    lib.smat_profile_table_element_bytes.argtypes = [vp]
    lib.smat_profile_table_element_bytes.restype = i
    lib.smat_uses_tensor_cores.argtypes = [vp]
    lib.smat_uses_tensor_cores.restype = i
    lib.smat_gated_forward_uses_tensor_cores.argtypes = [vp]
    lib.smat_gated_forward_uses_tensor_cores.restype = i
    lib.smat_gated_backward_uses_tensor_cores.argtypes = [vp]
    lib.smat_gated_backward_uses_tensor_cores.restype = i
    lib.smat_forward_causal_static.argtypes = [vp, vp, vp, vp, i, i, i64, vp]
    lib.smat_forward_causal_static.restype = i
    lib.smat_static_check_status.argtypes = [vp]
    lib.smat_static_check_status.restype = i
    lib.smat_debug_timeout_probe.argtypes = [vp, i64, vp]
    lib.smat_debug_timeout_probe.restype = i
    lib.smat_measure_fadd_rate.argtypes = [vp, i, ctypes.POINTER(ctypes.c_double), vp]
    lib.smat_measure_fadd_rate.restype = i
    lib.smat_profile_enable.argtypes = [vp, i]
    lib.smat_profile_enable.restype = i
    lib.smat_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_float), i]
    lib.smat_profile_read.restype = i
    lib.smat_status_string.argtypes = [i]
    lib.smat_status_string.restype = ctypes.c_char_p
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().smat_status_string(int(code)).decode()


def _check(code: int, what: str) -> None:
    if code != 0:
        raise SmatError(code, what)


def _ptr(t: torch.Tensor | None) -> int | None:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


_TORCH_DTYPE = {SMAT_F32: torch.float32, SMAT_BF16: torch.bfloat16}

STATIC_MAX_TILES = 1024


def forward_causal_static(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, O: torch.Tensor | None = None,
                          stream=None) -> torch.Tensor:
    """Causal (d = 1) forward that needs no workspace: smat_forward_causal_static.

    For callers that may not allocate device memory; the scratch lives in a fixed 32 MiB array inside the
    library, so batch * heads * T / 128 must not exceed STATIC_MAX_TILES, and calls must not overlap on the GPU.
    O may be passed in by a caller who cannot allocate; it is created here only as a convenience."""
    lib = load_library()
    for name, t in (("Q", Q), ("K", K), ("V", V)):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and t.dim() == 4 and t.shape[-1] == 128):
            raise ValueError(f"{name}: expected a contiguous CUDA bf16 tensor [batch, heads, T, 128]")
    if O is None:
        O = torch.empty_like(V)
    b, h, T, _ = Q.shape
    _check(lib.smat_forward_causal_static(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), b, h, T, _stream(stream)),
           "smat_forward_causal_static")
    return O


def static_check_status(stream=None) -> None:
    """Raises if the last forward_causal_static on this device hit a bounded-wait expiry (smat_static_check_status)."""
    _check(load_library().smat_static_check_status(_stream(stream)), "smat_static_check_status")


def debug_timeout_probe(workspace: torch.Tensor, limit_cycles: int = 2_000_000, stream=None) -> None:
    """smat_debug_timeout_probe: a wait that is meant to run out sets the status word of `workspace`."""
    _check(load_library().smat_debug_timeout_probe(_ptr(workspace), int(limit_cycles), _stream(stream)),
           "smat_debug_timeout_probe")


def measure_fadd_rate(packed: bool = False, stream=None) -> float:
    """fp32 additions per second of the plain ALUs, measured (smat_measure_fadd_rate)."""
    scratch = torch.zeros(64, dtype=torch.float32, device="cuda")
    out = ctypes.c_double(0.0)
    _check(load_library().smat_measure_fadd_rate(_ptr(scratch), int(packed), ctypes.byref(out), _stream(stream)),
           "smat_measure_fadd_rate")
    return float(out.value)


class SmatPlan:
    """Owns one smat_plan and (optionally) a workspace tensor; mirrors the C entry points."""

    def __init__(self, batch: int, heads: int, T: int, d_k: int, d_v: int, d: int, chunk: int, dtype="bf16",
                 q_override: int = 0, flags: int = 0):
        self.lib = load_library()
        self.dtype_code = {"f32": SMAT_F32, "bf16": SMAT_BF16}[dtype] if isinstance(dtype, str) else int(dtype)
        self.torch_dtype = _TORCH_DTYPE[self.dtype_code]
        self.shape = (batch, heads, T, d_k, d_v)
        self.flags = int(flags)
        handle = ctypes.c_void_p()
        _check(self.lib.smat_plan_create(ctypes.byref(handle), batch, heads, T, d_k, d_v, d, chunk, q_override,
                                         self.dtype_code, flags), "smat_plan_create")
        self.handle = handle
        self._ws = None

    def __del__(self):
        if getattr(self, "handle", None) and self.lib is not None:
            self.lib.smat_plan_destroy(self.handle)
            self.handle = None

    # -- queries ---------------------------------------------------------------------------
    def geometry(self) -> Geometry:
        g = _Geometry()
        _check(self.lib.smat_get_geometry(self.handle, ctypes.byref(g)), "smat_get_geometry")
        return Geometry(g.T, g.c, g.n, g.m, g.d, g.q, g.P, g.A, g.B, g.nnzC, bool(g.vc_conditions_met))

    def uses_tensor_cores(self) -> bool:
        return bool(self.lib.smat_uses_tensor_cores(self.handle))

    def gated_forward_uses_tensor_cores(self) -> bool:
        return bool(self.lib.smat_gated_forward_uses_tensor_cores(self.handle))

    def gated_backward_uses_tensor_cores(self) -> bool:
        return bool(self.lib.smat_gated_backward_uses_tensor_cores(self.handle))

    def type_table_element_bytes(self) -> int:
        return int(self.lib.smat_type_table_element_bytes(self.handle))

    def profile_table_element_bytes(self) -> int:
        return int(self.lib.smat_profile_table_element_bytes(self.handle))

    def workspace_bytes(self, for_backward: bool = False) -> int:
        return int(self.lib.smat_workspace_bytes(self.handle, int(for_backward)))

    def workspace(self, for_backward: bool = False, device="cuda") -> torch.Tensor:
        need = self.workspace_bytes(for_backward)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=device)
        return self._ws

    def profile_enable(self, enable: bool = True) -> None:
        _check(self.lib.smat_profile_enable(self.handle, int(enable)), "smat_profile_enable")

    def profile_read(self, max_stages: int = 64):
        """[(kernel name, milliseconds)] of the last forward/backward, in launch order."""
        names = (ctypes.c_char_p * max_stages)()
        ms = (ctypes.c_float * max_stages)()
        count = self.lib.smat_profile_read(self.handle, names, ms, max_stages)
        return [(names[k].decode(), float(ms[k])) for k in range(count)]

    def last_launch_count(self) -> int:
        return int(self.lib.smat_last_launch_count(self.handle))

    # -- the hot path ------------------------------------------------------------------------
    def _check_tensor(self, t: torch.Tensor, last: int, name: str) -> None:
        b, h, T, _, _ = self.shape
        if not t.is_cuda:
            raise ValueError(f"{name} must be a CUDA tensor")
        if t.dtype != self.torch_dtype or tuple(t.shape) != (b, h, T, last) or not t.is_contiguous():
            raise ValueError(f"{name}: expected contiguous {self.torch_dtype} of shape {(b, h, T, last)}, "
                             f"got {t.dtype} {tuple(t.shape)}")

    def _check_routing(self, prof, typ):
        b, h, _, _, _ = self.shape
        g = self.geometry()
        for name, t, count in (("prof", prof, g.n), ("type", typ, g.m)):
            if not (t.is_cuda and t.dtype == torch.int32 and t.is_contiguous() and tuple(t.shape) == (b * h, count)):
                raise ValueError(f"{name}: expected a contiguous CUDA int32 tensor of shape {(b * h, count)}")

    def forward(self, Q, K, V, O=None, workspace=None, stream=None, prof=None, type=None):
        """smat_forward, or smat_forward_routed when prof [batch*heads, n] and type [batch*heads, m] are given."""
        _, _, _, dk, dv = self.shape
        self._check_tensor(Q, dk, "Q"); self._check_tensor(K, dk, "K"); self._check_tensor(V, dv, "V")
        if O is None:
            O = torch.empty_like(V)
        self._check_tensor(O, dv, "O")
        ws = self.workspace(False, Q.device) if workspace is None else workspace
        if prof is not None or type is not None:
            self._check_routing(prof, type)
            _check(self.lib.smat_forward_routed(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(prof), _ptr(type),
                                                _ptr(ws), ws.numel(), _stream(stream)), "smat_forward_routed")
            return O
        _check(self.lib.smat_forward(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(ws), ws.numel(),
                                     _stream(stream)), "smat_forward")
        return O

    def backward(self, Q, K, V, dO, dQ=None, dK=None, dV=None, workspace=None, stream=None, prof=None, type=None):
        _, _, _, dk, dv = self.shape
        self._check_tensor(Q, dk, "Q"); self._check_tensor(K, dk, "K"); self._check_tensor(V, dv, "V")
        self._check_tensor(dO, dv, "dO")
        dQ = torch.empty_like(Q) if dQ is None else dQ
        dK = torch.empty_like(K) if dK is None else dK
        dV = torch.empty_like(V) if dV is None else dV
        ws = self.workspace(True, Q.device) if workspace is None else workspace
        if prof is not None or type is not None:
            self._check_routing(prof, type)
            _check(self.lib.smat_backward_routed(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(dQ), _ptr(dK),
                                                 _ptr(dV), _ptr(prof), _ptr(type), _ptr(ws), ws.numel(), _stream(stream)),
                   "smat_backward_routed")
            return dQ, dK, dV
        _check(self.lib.smat_backward(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(dO), _ptr(dQ), _ptr(dK), _ptr(dV),
                                      _ptr(ws), ws.numel(), _stream(stream)), "smat_backward")
        return dQ, dK, dV

    # -- normalised output ------------------------------------------------------------------------
    def forward_normalized(self, Q, K, V, O=None, workspace=None, stream=None):
        """V: p - 1 value columns and the normaliser column last; O: normalised values and the normaliser last."""
        _, _, _, dk, dv = self.shape
        self._check_tensor(Q, dk, "Q"); self._check_tensor(K, dk, "K"); self._check_tensor(V, dv, "V")
        O = torch.empty_like(V) if O is None else O
        ws = self.workspace(False, Q.device) if workspace is None else workspace
        _check(self.lib.smat_forward_normalized(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(ws), ws.numel(),
                                                _stream(stream)), "smat_forward_normalized")
        return O

    def backward_normalized(self, Q, K, V, O, dO, workspace=None, stream=None):
        _, _, _, dk, dv = self.shape
        self._check_tensor(Q, dk, "Q"); self._check_tensor(K, dk, "K"); self._check_tensor(V, dv, "V")
        self._check_tensor(O, dv, "O"); self._check_tensor(dO, dv, "dO")
        dQ, dK, dV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
        ws = self.workspace(True, Q.device) if workspace is None else workspace
        _check(self.lib.smat_backward_normalized(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(dO), _ptr(dQ),
                                                 _ptr(dK), _ptr(dV), _ptr(ws), ws.numel(), _stream(stream)),
               "smat_backward_normalized")
        return dQ, dK, dV

    # -- scalar-gated variant ---------------------------------------------------------------------
    def _check_gates(self, log_a):
        b, h, T, _, _ = self.shape
        if not (log_a.is_cuda and log_a.dtype == torch.float32 and log_a.is_contiguous() and tuple(log_a.shape) == (b * h, T)):
            raise ValueError(f"log_a: expected a contiguous CUDA float32 tensor of shape {(b * h, T)}")

    def forward_gated(self, Q, K, V, log_a, O=None, workspace=None, stream=None):
        _, _, _, dk, dv = self.shape
        self._check_tensor(Q, dk, "Q"); self._check_tensor(K, dk, "K"); self._check_tensor(V, dv, "V")
        self._check_gates(log_a)
        O = torch.empty_like(V) if O is None else O
        ws = self.workspace(False, Q.device) if workspace is None else workspace
        _check(self.lib.smat_forward_gated(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(log_a), _ptr(O), _ptr(ws),
                                           ws.numel(), _stream(stream)), "smat_forward_gated")
        return O

    def backward_gated(self, Q, K, V, log_a, dO, dQ=None, dK=None, dV=None, dlog_a=None, workspace=None, stream=None):
        _, _, _, dk, dv = self.shape
        self._check_tensor(Q, dk, "Q"); self._check_tensor(K, dk, "K"); self._check_tensor(V, dv, "V")
        self._check_tensor(dO, dv, "dO")
        self._check_gates(log_a)
        dQ = torch.empty_like(Q) if dQ is None else dQ
        dK = torch.empty_like(K) if dK is None else dK
        dV = torch.empty_like(V) if dV is None else dV
        dla = torch.empty_like(log_a) if dlog_a is None else dlog_a
        ws = self.workspace(True, Q.device) if workspace is None else workspace
        _check(self.lib.smat_backward_gated(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(log_a), _ptr(dO), _ptr(dQ),
                                            _ptr(dK), _ptr(dV), _ptr(dla), _ptr(ws), ws.numel(), _stream(stream)),
               "smat_backward_gated")
        return dQ, dK, dV, dla

    # -- cached decoding -----------------------------------------------------------------------
    def decode_cache(self, device="cuda") -> torch.Tensor:
        return torch.empty(int(self.lib.smat_decode_cache_bytes(self.handle)), dtype=torch.uint8, device=device)

    def decode_begin(self, K, V, cache, workspace=None, stream=None) -> None:
        _, _, _, dk, dv = self.shape
        self._check_tensor(K, dk, "K"); self._check_tensor(V, dv, "V")
        ws = self.workspace(False, K.device) if workspace is None else workspace
        self._ws = ws
        _check(self.lib.smat_decode_begin(self.handle, _ptr(K), _ptr(V), _ptr(cache), cache.numel(), _ptr(ws), ws.numel(),
                                          _stream(stream)), "smat_decode_begin")

    def decode_step(self, q, k, v, t: int, cache, o=None, stream=None):
        b, h, _, dk, dv = self.shape
        for name, x, dim in (("q", q, dk), ("k", k, dk), ("v", v, dv)):
            if not (x.is_cuda and x.is_contiguous() and x.dtype == self.torch_dtype and tuple(x.shape) == (b, h, dim)):
                raise ValueError(f"{name}: expected a contiguous CUDA tensor [{b}, {h}, {dim}] of the plan's dtype")
        o = torch.empty_like(v) if o is None else o
        _check(self.lib.smat_decode_step(self.handle, _ptr(q), _ptr(k), _ptr(v), int(t), _ptr(o), _ptr(cache), cache.numel(),
                                         _stream(stream)), "smat_decode_step")
        return o

    def decode_begin_gated(self, K, V, log_a, cache, workspace=None, stream=None) -> None:
        _, _, _, dk, dv = self.shape
        self._check_tensor(K, dk, "K"); self._check_tensor(V, dv, "V")
        self._check_gates(log_a)
        ws = self.workspace(False, K.device) if workspace is None else workspace
        self._ws = ws
        _check(self.lib.smat_decode_begin_gated(self.handle, _ptr(K), _ptr(V), _ptr(log_a), _ptr(cache), cache.numel(),
                                                _ptr(ws), ws.numel(), _stream(stream)), "smat_decode_begin_gated")

    def decode_step_gated(self, q, k, v, log_a_t, t: int, cache, o=None, stream=None):
        b, h, _, dk, dv = self.shape
        for name, x, dim in (("q", q, dk), ("k", k, dk), ("v", v, dv)):
            if not (x.is_cuda and x.is_contiguous() and x.dtype == self.torch_dtype and tuple(x.shape) == (b, h, dim)):
                raise ValueError(f"{name}: expected a contiguous CUDA tensor [{b}, {h}, {dim}] of the plan's dtype")
        if not (log_a_t.is_cuda and log_a_t.is_contiguous() and log_a_t.dtype == torch.float32 and log_a_t.numel() == b * h):
            raise ValueError(f"log_a_t: expected a contiguous CUDA fp32 tensor of {b * h} log-gates")
        o = torch.empty_like(v) if o is None else o
        _check(self.lib.smat_decode_step_gated(self.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(log_a_t), int(t), _ptr(o),
                                               _ptr(cache), cache.numel(), _stream(stream)), "smat_decode_step_gated")
        return o

    # -- verification exports ------------------------------------------------------------------
    def routing_indices(self):
        g = self.geometry()
        D = max(g.d - 1, 0)
        prof = torch.zeros((g.n, D), dtype=torch.int32)
        typ = torch.zeros(g.m, dtype=torch.int32)
        ab = torch.zeros((g.B, g.d), dtype=torch.int32)
        _check(self.lib.smat_routing_indices(self.handle, _ptr(prof) if prof.numel() else None, _ptr(typ), _ptr(ab)),
               "smat_routing_indices")
        return prof, typ, ab

    def debug_mask(self, device="cuda", stream=None) -> torch.Tensor:
        T = self.shape[2]
        mask = torch.empty((T, T), dtype=torch.uint8, device=device)
        _check(self.lib.smat_debug_mask(self.handle, _ptr(mask), _stream(stream)), "smat_debug_mask")
        return mask

    def debug_tables(self, workspace=None, stream=None):
        b, h, T, dk, dv = self.shape
        g = self.geometry()
        ws = self._ws if workspace is None else workspace
        tc = self.uses_tensor_cores()
        tiles = tc and bool(self.flags & FLAG_PER_TILE_STATES)   # per-tile states exist on tensor-core plans only then
        F = U = Sin = None
        if not (tc and g.d == 1 and not tiles):
            F = torch.empty((b * h, g.P, dk, dv), dtype=torch.float32, device=ws.device)
            U = torch.empty((b * h, g.B, dk, dv), dtype=torch.float32, device=ws.device)
        if not tc or tiles:
            Sin = torch.empty((b * h, T // (128 if tc else g.c), dk, dv), dtype=torch.float32, device=ws.device)
        _check(self.lib.smat_debug_tables(self.handle, _ptr(ws), _ptr(F), _ptr(U), _ptr(Sin), _stream(stream)),
               "smat_debug_tables")
        return F, U, Sin

    def check_status(self, workspace=None, stream=None) -> None:
        ws = self._ws if workspace is None else workspace
        _check(self.lib.smat_check_status(self.handle, _ptr(ws), _stream(stream)), "smat_check_status")
