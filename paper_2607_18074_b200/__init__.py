"""Thin Python binding of libsobek (argument marshalling only).

Every step of the convolution runs in the library's CUDA kernels; torch is used for device
memory and streams.  There is no fallback: if the shared library is missing or a call
fails, an exception is raised.

Names mirror the C ABI (include/sobek.h): `Plan` <-> sobek_plan_*, `graph_prepare`,
`workspace_bytes`, `conv_fwd`, `conv_bwd`, `conv_dbwd`, `last_device_status`.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, byref, c_char_p, c_double, c_float, c_int, c_int32, c_int64, c_size_t, c_uint, c_uint32, c_void_p

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsobek.so")

FLAG_UVU = 1      # SOBEK_FLAG_UVU: channelwise multiplicity mode
FLAG_MUL_IR = 2   # SOBEK_FLAG_MUL_IR: node features cross the boundary in mul_ir order
FLAG_FAST_GEMM = 4  # SOBEK_FLAG_FAST_GEMM: node-side GEMMs as plain bf16 products (optional, lower precision)
FLAG_FUSED_FP32 = 8    # SOBEK_FLAG_FUSED_FP32: fused FP32-pipe stream + contraction schedule
FLAG_FP32_STREAM = 16  # SOBEK_FLAG_FP32_STREAM: edge stream on the FP32 pipes
FLAG_FP32_EDGE = 32    # SOBEK_FLAG_FP32_EDGE: edge pass on the FP32 pipes
FLAG_UVU_STATE = 64        # SOBEK_FLAG_UVU_STATE: channelwise y and gx through the receiver state


def flag_state_budget_mib(mb: int) -> int:
    """SOBEK_FLAG_STATE_BUDGET_MIB: the scratch budget in MiB, carried in bits 12..31 of the flags word."""
    if not 1 <= int(mb) < (1 << 20):
        raise ValueError(mb)
    return int(mb) << 12

EXPORTS = [
    "sobek_plan_create", "sobek_plan_destroy", "sobek_plan_info", "sobek_plan_path", "sobek_plan_cg",
    "sobek_graph_prepare_bytes", "sobek_graph_prepare", "sobek_graph_receivers", "sobek_workspace_bytes", "sobek_conv_fwd",
    "sobek_conv_bwd", "sobek_conv_dbwd", "sobek_last_device_status", "sobek_status_string",
    "sobek_launch_count", "sobek_timing_enable", "sobek_timing_classes", "sobek_timing_class_name",
    "sobek_timing_collect", "sobek_static_scratch_bytes", "sobek_conv_fwd_static", "sobek_selftest_wait_timeout",
    "sobek_conv_fwd_retain", "sobek_conv_bwd_retained", "sobek_static_last_status", "sobek_measure_fp32_peak",
    "sobek_edge_vectors", "sobek_conv_geo_fwd", "sobek_conv_geo_bwd", "sobek_conv_geo_dbwd", "sobek_position_gradient",
    "sobek_geo_dbwd_full_workspace_bytes", "sobek_conv_geo_dbwd_full",
]
BASIS_BESSEL, BASIS_GAUSSIAN = 0, 1


class SobekError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


class Irrep(Structure):
    _fields_ = [("mul", c_int32), ("l", c_int32), ("parity", c_int32)]


class Info(Structure):
    _fields_ = [("C_x", c_int32), ("C_y", c_int32), ("dim_sh", c_int32), ("K", c_int32),
                ("n_paths", c_int32), ("l_max", c_int32), ("N_w", c_int64),
                ("state_floats_fwd", c_int64), ("state_floats_bwd", c_int64)]


class PathInfo(Structure):
    _fields_ = [("i_in", c_int32), ("l_sh", c_int32), ("i_out", c_int32), ("l_in", c_int32),
                ("l_out", c_int32), ("c_in", c_int32), ("c_out", c_int32), ("in_off", c_int32),
                ("sh_off", c_int32), ("out_off", c_int32), ("w_off", c_int64)]


class Graph(Structure):
    _fields_ = [("N", c_int64), ("E", c_int64), ("row_ptr", c_void_p), ("col", c_void_p),
                ("src_ptr", c_void_p), ("src_perm", c_void_p), ("src_recv", c_void_p)]


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with "
                              "`python -m paper_2607_18074_b200.build` (needs nvcc)")
        L = ctypes.CDLL(LIB_PATH)
        L.sobek_plan_create.argtypes = [POINTER(Irrep), c_int, POINTER(Irrep), c_int, c_int, c_int,
                                        c_uint32, POINTER(c_void_p)]
        L.sobek_plan_destroy.argtypes = [c_void_p]
        L.sobek_plan_destroy.restype = None
        L.sobek_plan_info.argtypes = [c_void_p, POINTER(Info)]
        L.sobek_plan_path.argtypes = [c_void_p, c_int, POINTER(PathInfo)]
        L.sobek_plan_cg.argtypes = [c_void_p, c_int, POINTER(c_double)]
        L.sobek_graph_prepare_bytes.argtypes = [c_int64, c_int64]
        L.sobek_graph_prepare_bytes.restype = c_size_t
        L.sobek_graph_prepare.argtypes = [c_int64, c_int64] + [c_void_p] * 5 + [c_size_t, c_void_p]
        L.sobek_graph_receivers.argtypes = [c_int64, c_int64] + [c_void_p] * 4
        L.sobek_workspace_bytes.argtypes = [c_void_p, c_int64, c_int64, c_int]
        L.sobek_workspace_bytes.restype = c_size_t
        L.sobek_conv_fwd.argtypes = [c_void_p, POINTER(Graph)] + [c_void_p] * 6 + [c_size_t, c_void_p]
        L.sobek_conv_bwd.argtypes = [c_void_p, POINTER(Graph)] + [c_void_p] * 10 + [c_size_t, c_void_p]
        L.sobek_conv_dbwd.argtypes = [c_void_p, POINTER(Graph)] + [c_void_p] * 15 + [c_size_t, c_void_p]
        L.sobek_conv_fwd_retain.argtypes = [c_void_p, POINTER(Graph)] + [c_void_p] * 6 + [c_size_t, c_void_p, POINTER(c_int)]
        L.sobek_conv_bwd_retained.argtypes = [c_void_p, POINTER(Graph)] + [c_void_p] * 10 + [c_size_t, c_void_p, c_int]
        L.sobek_edge_vectors.argtypes = [POINTER(Graph), c_void_p, c_void_p, c_void_p]
        L.sobek_position_gradient.argtypes = [POINTER(Graph), c_void_p, c_void_p, c_void_p]
        L.sobek_conv_geo_fwd.argtypes = [c_void_p, POINTER(Graph), c_void_p, c_int, c_float, c_int] + [c_void_p] * 4 + [c_size_t, c_void_p]
        L.sobek_conv_geo_bwd.argtypes = [c_void_p, POINTER(Graph), c_void_p, c_int, c_float, c_int] + [c_void_p] * 7 + [c_size_t, c_void_p]
        L.sobek_conv_geo_dbwd.argtypes = [c_void_p, POINTER(Graph), c_void_p, c_int, c_float, c_int] + [c_void_p] * 10 + [c_size_t, c_void_p]
        L.sobek_conv_geo_dbwd_full.argtypes = [c_void_p, POINTER(Graph), c_void_p, c_int, c_float, c_int] + [c_void_p] * 11 + [c_size_t, c_void_p]
        L.sobek_geo_dbwd_full_workspace_bytes.argtypes = [c_void_p, c_int64, c_int64]
        L.sobek_geo_dbwd_full_workspace_bytes.restype = c_size_t
        L.sobek_selftest_wait_timeout.argtypes = [c_void_p, c_uint, c_void_p]
        L.sobek_last_device_status.argtypes = [c_void_p, c_void_p]
        L.sobek_static_scratch_bytes.restype = c_size_t
        L.sobek_conv_fwd_static.argtypes = [c_void_p, POINTER(Graph)] + [c_void_p] * 6
        L.sobek_static_last_status.argtypes = [c_void_p]
        L.sobek_measure_fp32_peak.argtypes = [c_double, c_void_p, c_size_t, POINTER(c_double), c_void_p]
        L.sobek_status_string.argtypes = [c_int]
        L.sobek_status_string.restype = c_char_p
        L.sobek_launch_count.restype = c_int64
        L.sobek_timing_enable.argtypes = [c_int]
        L.sobek_timing_class_name.argtypes = [c_int]
        L.sobek_timing_class_name.restype = c_char_p
        L.sobek_timing_collect.argtypes = [POINTER(c_double), POINTER(c_int64)]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().sobek_status_string(int(code)).decode()


def launch_count() -> int:
    return int(lib().sobek_launch_count())


def timing_enable(on: bool):
    lib().sobek_timing_enable(1 if on else 0)


def timing_collect():
    """{kernel class: (total device ms, launches)} since timing was enabled / last collected."""
    n = lib().sobek_timing_classes()
    ms, cnt = (c_double * n)(), (c_int64 * n)()
    _check(lib().sobek_timing_collect(ms, cnt), "sobek_timing_collect")
    return {lib().sobek_timing_class_name(k).decode(): (ms[k], cnt[k]) for k in range(n)}


def _check(code, where):
    if code != 0:
        raise SobekError(code, where)


def _irreps(seq):
    arr = (Irrep * len(seq))()
    for k, (mul, l, p) in enumerate(seq):
        arr[k] = Irrep(mul, l, p)
    return arr


class Plan:
    """sobek_plan: irreps are sequences of (mul, l, parity) with parity +1 / -1.  mode "uvw" is the fully
    connected multiplicity mixing, "uvu" the channelwise one (SOBEK_FLAG_UVU).  layout "ir_mul" (block offset +
    m*mul + u) is the kernels' own order of node features, "mul_ir" (block offset + u*(2l+1) + m) is transposed at the
    boundary (SOBEK_FLAG_MUL_IR).  fused / tc_stream / tc_edge / state_budget_mib map to SOBEK_FLAG_FUSED_FP32,
    SOBEK_FLAG_FP32_STREAM, SOBEK_FLAG_FP32_EDGE and SOBEK_FLAG_STATE_BUDGET_MIB; uvu_state to
    SOBEK_FLAG_UVU_STATE (channelwise y and gx through the receiver state even where the direct kernel applies)."""

    def __init__(self, irreps_in, irreps_out, l_max: int, K: int, flags: int = 0, mode: str = "uvw",
                 layout: str = "ir_mul", fused: bool = False, tc_stream: bool = True, tc_edge: bool = True,
                 state_budget_mib: int | None = None, uvu_state: bool = False):
        if mode not in ("uvw", "uvu"):
            raise ValueError(mode)
        if layout not in ("ir_mul", "mul_ir"):
            raise ValueError(layout)
        if mode == "uvu":
            flags |= FLAG_UVU
        if layout == "mul_ir":
            flags |= FLAG_MUL_IR
        if fused:
            flags |= FLAG_FUSED_FP32
        if not tc_stream:
            flags |= FLAG_FP32_STREAM
        if not tc_edge:
            flags |= FLAG_FP32_EDGE
        if state_budget_mib is not None:
            flags |= flag_state_budget_mib(state_budget_mib)
        if uvu_state:
            flags |= FLAG_UVU_STATE
        self.layout = "mul_ir" if flags & FLAG_MUL_IR else "ir_mul"
        self.mode = "uvu" if flags & FLAG_UVU else "uvw"
        self._h = c_void_p()
        a, b = _irreps(irreps_in), _irreps(irreps_out)
        _check(lib().sobek_plan_create(a, len(irreps_in), b, len(irreps_out), l_max, K, flags,
                                       byref(self._h)), "sobek_plan_create")
        self.info = Info()
        _check(lib().sobek_plan_info(self._h, byref(self.info)), "sobek_plan_info")

    def __del__(self):
        h = getattr(self, "_h", None)
        if h and _lib is not None:
            _lib.sobek_plan_destroy(h)
            self._h = None

    @property
    def handle(self):
        return self._h

    def path(self, k: int) -> PathInfo:
        pi = PathInfo()
        _check(lib().sobek_plan_path(self._h, k, byref(pi)), "sobek_plan_path")
        return pi

    def cg(self, k: int):
        import numpy as np
        pi = self.path(k)
        shape = (2 * pi.l_in + 1, 2 * pi.l_sh + 1, 2 * pi.l_out + 1)
        out = np.zeros(shape, dtype=np.float64)
        _check(lib().sobek_plan_cg(self._h, k, out.ctypes.data_as(POINTER(c_double))), "sobek_plan_cg")
        return out


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream():
    import torch
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def graph_prepare_bytes(N: int, E: int) -> int:
    return int(lib().sobek_graph_prepare_bytes(N, E))


def graph_prepare(row_ptr, col):
    """Validates the receiver-sorted CSR (int64 row_ptr[N+1], int32 col[E], CUDA tensors) and
    returns the sender-sorted view (src_ptr int64[N+1], src_perm int32[E])."""
    import torch
    N, E = row_ptr.numel() - 1, col.numel()
    src_ptr = torch.empty(N + 1, dtype=torch.int64, device=row_ptr.device)
    src_perm = torch.empty(E, dtype=torch.int32, device=row_ptr.device)
    nbytes = graph_prepare_bytes(N, E)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=row_ptr.device)
    _check(lib().sobek_graph_prepare(N, E, _ptr(row_ptr), _ptr(col), _ptr(src_ptr), _ptr(src_perm),
                                     _ptr(ws), nbytes, _stream()), "sobek_graph_prepare")
    return src_ptr, src_perm


def graph_receivers(row_ptr, src_perm):
    """src_recv int32[E]: the receiver of edge src_perm[p] at every position p of the sender-sorted view."""
    import torch
    N, E = row_ptr.numel() - 1, src_perm.numel()
    src_recv = torch.empty(E, dtype=torch.int32, device=row_ptr.device)
    _check(lib().sobek_graph_receivers(N, E, _ptr(row_ptr), _ptr(src_perm), _ptr(src_recv), _stream()),
           "sobek_graph_receivers")
    return src_recv


def make_graph(row_ptr, col, src_ptr=None, src_perm=None, src_recv=None) -> Graph:
    """The sobek_graph descriptor of five CUDA tensors.  The descriptor holds raw device addresses, so the
    returned object also keeps references to the tensors: they stay allocated for as long as it lives."""
    g = Graph(row_ptr.numel() - 1, col.numel(), _ptr(row_ptr), _ptr(col), _ptr(src_ptr), _ptr(src_perm),
              _ptr(src_recv))
    g.tensors = (row_ptr, col, src_ptr, src_perm, src_recv)
    return g


def workspace_bytes(plan: Plan, N: int, E: int, order: int) -> int:
    return int(lib().sobek_workspace_bytes(plan.handle, N, E, order))


def conv_fwd(plan, graph, x, Y, phi, R, y, ws):
    _check(lib().sobek_conv_fwd(plan.handle, byref(graph), _ptr(x), _ptr(Y), _ptr(phi), _ptr(R), _ptr(y),
                                _ptr(ws), ws.numel() * ws.element_size(), _stream()), "sobek_conv_fwd")


def static_scratch_bytes() -> int:
    return int(lib().sobek_static_scratch_bytes())


def conv_fwd_static(plan, graph, x, Y, phi, R, y):
    """Forward convolution without a workspace: for callers that cannot allocate device memory
    when they run the operator.  Scratch lives in a fixed 32 MiB array inside the library (see
    sobek_conv_fwd_static in include/sobek.h for the size limit and the sharing rules)."""
    _check(lib().sobek_conv_fwd_static(plan.handle, byref(graph), _ptr(x), _ptr(Y), _ptr(phi), _ptr(R),
                                       _ptr(y), _stream()), "sobek_conv_fwd_static")


def static_last_status() -> int:
    """Status word left by the kernels of the last conv_fwd_static call on the current device (synchronises)."""
    return int(lib().sobek_static_last_status(_stream()))


def conv_bwd(plan, graph, x, Y, phi, R, gy, gx, gY, gphi, gR, ws):
    _check(lib().sobek_conv_bwd(plan.handle, byref(graph), _ptr(x), _ptr(Y), _ptr(phi), _ptr(R), _ptr(gy),
                                _ptr(gx), _ptr(gY), _ptr(gphi), _ptr(gR), _ptr(ws),
                                ws.numel() * ws.element_size(), _stream()), "sobek_conv_bwd")


def edge_vectors(graph, pos, rvec):
    _check(lib().sobek_edge_vectors(byref(graph), _ptr(pos), _ptr(rvec), _stream()), "sobek_edge_vectors")


def position_gradient(graph, g_rvec, gpos):
    _check(lib().sobek_position_gradient(byref(graph), _ptr(g_rvec), _ptr(gpos), _stream()), "sobek_position_gradient")


def conv_geo_fwd(plan, graph, rvec, basis, r_cut, envelope_p, x, R, y, ws):
    _check(lib().sobek_conv_geo_fwd(plan.handle, byref(graph), _ptr(rvec), int(basis), float(r_cut), int(envelope_p),
                                    _ptr(x), _ptr(R), _ptr(y), _ptr(ws), ws.numel() * ws.element_size(), _stream()),
           "sobek_conv_geo_fwd")


def conv_geo_bwd(plan, graph, rvec, basis, r_cut, envelope_p, x, R, gy, gx, g_rvec, gR, ws):
    _check(lib().sobek_conv_geo_bwd(plan.handle, byref(graph), _ptr(rvec), int(basis), float(r_cut), int(envelope_p),
                                    _ptr(x), _ptr(R), _ptr(gy), _ptr(gx), _ptr(g_rvec), _ptr(gR), _ptr(ws),
                                    ws.numel() * ws.element_size(), _stream()), "sobek_conv_geo_bwd")


def conv_geo_dbwd(plan, graph, rvec, basis, r_cut, envelope_p, x, R, gy, vx, v_rvec, vR, ggy, hx, hR, ws):
    _check(lib().sobek_conv_geo_dbwd(plan.handle, byref(graph), _ptr(rvec), int(basis), float(r_cut), int(envelope_p),
                                     _ptr(x), _ptr(R), _ptr(gy), _ptr(vx), _ptr(v_rvec), _ptr(vR), _ptr(ggy), _ptr(hx),
                                     _ptr(hR), _ptr(ws), ws.numel() * ws.element_size(), _stream()), "sobek_conv_geo_dbwd")


def geo_dbwd_full_workspace_bytes(plan, N: int, E: int) -> int:
    return int(lib().sobek_geo_dbwd_full_workspace_bytes(plan.handle, int(N), int(E)))


def conv_geo_dbwd_full(plan, graph, rvec, basis, r_cut, envelope_p, x, R, gy, vx, v_rvec, vR, ggy, hx, hR, h_rvec, ws):
    """sobek_conv_geo_dbwd_full: the outputs of conv_geo_dbwd plus h_rvec [E, 3]; ws of geo_dbwd_full_workspace_bytes."""
    _check(lib().sobek_conv_geo_dbwd_full(plan.handle, byref(graph), _ptr(rvec), int(basis), float(r_cut), int(envelope_p),
                                          _ptr(x), _ptr(R), _ptr(gy), _ptr(vx), _ptr(v_rvec), _ptr(vR), _ptr(ggy),
                                          _ptr(hx), _ptr(hR), _ptr(h_rvec), _ptr(ws), ws.numel() * ws.element_size(),
                                          _stream()), "sobek_conv_geo_dbwd_full")


def conv_fwd_retain(plan, graph, x, Y, phi, R, y, ws) -> int:
    """sobek_conv_fwd_retain: forward on an order-1 workspace; returns 1 if the state of all receivers stays in ws."""
    from ctypes import c_int
    kept = c_int(0)
    _check(lib().sobek_conv_fwd_retain(plan.handle, byref(graph), _ptr(x), _ptr(Y), _ptr(phi), _ptr(R), _ptr(y),
                                       _ptr(ws), ws.numel() * ws.element_size(), _stream(), byref(kept)),
           "sobek_conv_fwd_retain")
    return int(kept.value)


def conv_bwd_retained(plan, graph, x, Y, phi, R, gy, gx, gY, gphi, gR, ws, retained: int):
    _check(lib().sobek_conv_bwd_retained(plan.handle, byref(graph), _ptr(x), _ptr(Y), _ptr(phi), _ptr(R), _ptr(gy),
                                         _ptr(gx), _ptr(gY), _ptr(gphi), _ptr(gR), _ptr(ws),
                                         ws.numel() * ws.element_size(), _stream(), int(retained)),
           "sobek_conv_bwd_retained")


def conv_dbwd(plan, graph, x, Y, phi, R, gy, vx, vY, vphi, vR, ggy, hx, hY, hphi, hR, ws):
    _check(lib().sobek_conv_dbwd(plan.handle, byref(graph), _ptr(x), _ptr(Y), _ptr(phi), _ptr(R), _ptr(gy),
                                 _ptr(vx), _ptr(vY), _ptr(vphi), _ptr(vR), _ptr(ggy), _ptr(hx), _ptr(hY),
                                 _ptr(hphi), _ptr(hR), _ptr(ws), ws.numel() * ws.element_size(),
                                 _stream()), "sobek_conv_dbwd")


def measure_fp32_peak(seconds: float = 1.0) -> float:
    """Sustained FP32 multiply-add rate of the current device in TFLOP/s (sobek_measure_fp32_peak)."""
    import torch
    n = 8192 * torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    scratch = torch.empty(n, dtype=torch.float32, device="cuda")
    out = c_double(0.0)
    _check(lib().sobek_measure_fp32_peak(float(seconds), _ptr(scratch), n, byref(out), _stream()),
           "sobek_measure_fp32_peak")
    return float(out.value)


def selftest_wait_timeout(ws, limit_ms: int = 200):
    """Enqueue the bounded-wait self-test; read its result with last_device_status(ws)."""
    _check(lib().sobek_selftest_wait_timeout(_ptr(ws), int(limit_ms), _stream()), "sobek_selftest_wait_timeout")


def last_device_status(ws) -> int:
    return int(lib().sobek_last_device_status(_ptr(ws), _stream()))
