"""ctypes binding of libfcp.so: same names as the C ABI in include/fcp.h, argument marshalling only.

Every step of the path runs inside the library's kernels; PyTorch is used by callers for device
memory and streams.  There is no fallback: if the shared library is missing, `lib()` raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfcp.so")

FCP_OK = 0
FCP_ERR_INVALID_ARG, FCP_ERR_INFEASIBLE, FCP_ERR_UNSUPPORTED, FCP_ERR_WORKSPACE = -1, -2, -3, -4
FCP_ERR_CUDA, FCP_ERR_TIMEOUT, FCP_ERR_NOT_UPLOADED = -5, -6, -7
FCP_MAX_DEGREE = 64

TABLES = dict(cu_seqlens=0, chunk_offset=1, chunk_bounds=2, pairs=3, items=4, slot_offset=5, slot_rows=6,
              fwd_units=7, bwd_units=8, bwd_qranges=9, merge_units=10, bwd_work=11, fused_units=12, row_limit=13,
              first_query=14, span_pairs=15)
_TABLE_WIDTH = dict(pairs=6, items=8, fwd_units=16, bwd_units=8, bwd_qranges=4, merge_units=4, fused_units=16,
                    span_pairs=5)
INFO = dict(T=0, R=1, n_pairs=2, n_items=3, n_fwd_units=4, n_bwd_units=5, n_merge_units=6, B=7, n_merge_multi=8,
            n_fused_units=9)

EXPORTS = ["fcp_plan_strategy", "fcp_plan_blocks", "fcp_plan_blocks_spans", "fcp_span_mask_efficiency", "fcp_plan_get", "fcp_plan_info", "fcp_plan_workspace_bytes",
           "fcp_plan_bwd_scratch_bytes", "fcp_plan_upload", "fcp_plan_destroy", "fcp_attn_fwd", "fcp_attn_fwd_merged",
           "fcp_attn_fwd_fused", "fcp_lse_merge", "fcp_attn_bwd", "fcp_attn_bwd_heads",
           "fcp_host_workspace_bytes", "fcp_attn_fwd_bwd_host", "fcp_last_device_status", "fcp_plan_set_profiling",
           "fcp_plan_kernel_ms", "fcp_noalloc_bytes_needed", "fcp_attn_bwd_noalloc", "fcp_noalloc_device_status",
           "fcp_selftest_bounded_wait", "fcp_status_string",
           "fcp_last_error_message"]


class FcpParams(C.Structure):
    _fields_ = [("hq", C.c_int32), ("hkv", C.c_int32), ("head_dim", C.c_int32), ("scale", C.c_float)]


class FcpCostCoeffs(C.Structure):
    _fields_ = [("alpha1", C.c_double), ("alpha2", C.c_double), ("alpha3", C.c_double), ("beta1", C.c_double),
                ("beta2", C.c_double), ("v", C.c_double), ("eta", C.POINTER(C.c_double))]


class FcpError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{status_string(status)}: {message}")
        self.status = status


_lib = None


def lib() -> C.CDLL:
    """Loads libfcp.so (built by paper_2602_21788_b200/build.py).  Raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} is missing: run `python -m paper_2602_21788_b200.build` (needs nvcc)")
    L = C.CDLL(LIB_PATH)
    i32p, i64p, f32p, f64p, vp = (C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.POINTER(C.c_float),
                                  C.POINTER(C.c_double), C.c_void_p)
    L.fcp_plan_strategy.argtypes = [i32p, C.c_int32, C.c_int32, C.c_double, C.c_double, C.c_double,
                                    C.POINTER(FcpCostCoeffs), i32p, i32p, i32p, f64p]
    L.fcp_plan_blocks.argtypes = [i32p, i32p, C.c_int32, C.POINTER(FcpParams), C.POINTER(vp)]
    L.fcp_plan_blocks_spans.argtypes = [i32p, i32p, C.c_int32, i32p, i32p, C.POINTER(FcpParams), C.POINTER(vp)]
    L.fcp_span_mask_efficiency.argtypes = [C.c_int32, i32p, C.c_int32, f64p]
    L.fcp_plan_get.argtypes = [vp, C.c_int32, C.POINTER(i32p), i64p]
    L.fcp_plan_info.argtypes = [vp, C.c_int32, i64p]
    L.fcp_plan_workspace_bytes.argtypes = [vp, C.c_int32, i64p, i64p, i64p]
    L.fcp_plan_upload.argtypes = [vp, vp]
    L.fcp_plan_destroy.argtypes = [vp]
    L.fcp_attn_fwd.argtypes = [vp, vp, vp, vp, C.c_int32, C.c_int32, vp, vp, vp]
    L.fcp_lse_merge.argtypes = [vp, vp, vp, C.c_int32, C.c_int32, vp, vp, vp, vp]
    L.fcp_attn_fwd_merged.argtypes = [vp, vp, vp, vp, C.c_int32, C.c_int32, vp, vp, vp, vp, vp]
    L.fcp_plan_set_profiling.argtypes = [vp, C.c_int32]
    L.fcp_plan_kernel_ms.argtypes = [vp, C.c_int32, i32p, f32p]
    L.fcp_attn_bwd.argtypes = [vp] * 11 + [C.c_int64, vp]
    L.fcp_attn_bwd_heads.argtypes = [vp] * 7 + [C.c_int32, C.c_int32] + [vp] * 4 + [C.c_int64, vp]
    L.fcp_attn_fwd_fused.argtypes = [vp, vp, vp, vp, C.c_int32, C.c_int32, vp, vp, vp, vp]
    L.fcp_plan_bwd_scratch_bytes.argtypes = [vp, C.c_int32, i64p]
    L.fcp_host_workspace_bytes.argtypes = [vp, i64p]
    L.fcp_attn_fwd_bwd_host.argtypes = [vp] * 11 + [C.c_int64, vp]
    L.fcp_last_device_status.argtypes = [vp, i32p]
    L.fcp_noalloc_bytes_needed.argtypes = [vp, i64p]
    L.fcp_attn_bwd_noalloc.argtypes = [vp] * 11
    L.fcp_noalloc_device_status.argtypes = [i32p]
    L.fcp_selftest_bounded_wait.argtypes = [C.c_uint32, i32p, vp]
    L.fcp_status_string.argtypes = [C.c_int]
    L.fcp_status_string.restype = C.c_char_p
    L.fcp_last_error_message.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("fcp_status_string", "fcp_last_error_message"):
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().fcp_status_string(int(status)).decode()


def _check(rc: int):
    if rc != FCP_OK:
        raise FcpError(rc, lib().fcp_last_error_message().decode())


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(C.POINTER(C.c_int32))


def _ptr(x):
    """Raw address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return C.c_void_p(x)
    if isinstance(x, np.ndarray):
        return C.c_void_p(x.ctypes.data)
    return C.c_void_p(x.data_ptr())


def fcp_plan_strategy(seqlens, N, E, M_token, M_ms, coeffs: dict, eta=None):
    """Returns dict(group_of, cp_degree, n_groups, makespan).  coeffs: alpha1..beta2, v."""
    sl, slp = _i32(seqlens)
    B = len(sl)
    eta_arr = None if eta is None else np.ascontiguousarray(eta, dtype=np.float64)
    cc = FcpCostCoeffs(coeffs["alpha1"], coeffs["alpha2"], coeffs["alpha3"], coeffs["beta1"], coeffs["beta2"],
                       coeffs["v"], None if eta_arr is None else eta_arr.ctypes.data_as(C.POINTER(C.c_double)))
    group_of = np.zeros(max(B, 1), dtype=np.int32)
    deg = np.zeros(max(B, 1), dtype=np.int32)
    ng = C.c_int32(0)
    mk = C.c_double(0.0)
    _check(lib().fcp_plan_strategy(slp, B, int(N), float(E), float(M_token), float(M_ms), C.byref(cc),
                                   group_of.ctypes.data_as(C.POINTER(C.c_int32)),
                                   deg.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(ng), C.byref(mk)))
    return dict(group_of=group_of[:B], cp_degree=deg[:B], n_groups=ng.value, makespan=mk.value)


class Plan:
    """Owns an fcp_plan handle."""

    def __init__(self, seqlens, cp_degrees, hq, hkv, head_dim, scale=0.0, spans=None):
        """spans: None, or one list of (begin, end) pairs per sequence (positions relative to its start)."""
        sl, slp = _i32(seqlens)
        dg, dgp = _i32(cp_degrees)
        if len(sl) != len(dg):
            raise ValueError("seqlens and cp_degrees differ in length")
        self.params = FcpParams(int(hq), int(hkv), int(head_dim), float(scale))
        self.handle = C.c_void_p()
        if spans is None:
            _check(lib().fcp_plan_blocks(slp, dgp, len(sl), C.byref(self.params), C.byref(self.handle)))
        else:
            if len(spans) != len(sl):
                raise ValueError("spans needs one list per sequence")
            off = np.zeros(len(sl) + 1, dtype=np.int32)
            off[1:] = np.cumsum([len(x) for x in spans])
            flat = np.asarray([v for x in spans for ab in x for v in ab], dtype=np.int32)
            so, sop = _i32(off)
            fl, flp = _i32(flat if flat.size else np.zeros(2, dtype=np.int32))
            _check(lib().fcp_plan_blocks_spans(slp, dgp, len(sl), sop, flp, C.byref(self.params), C.byref(self.handle)))
        self.hq, self.hkv, self.head_dim = int(hq), int(hkv), int(head_dim)

    def __del__(self):
        h = getattr(self, "handle", None)
        if h is not None and h.value and _lib is not None:
            _lib.fcp_plan_destroy(h)
            self.handle = None

    def table(self, name: str) -> np.ndarray:
        p = C.POINTER(C.c_int32)()
        n = C.c_int64(0)
        _check(lib().fcp_plan_get(self.handle, TABLES[name], C.byref(p), C.byref(n)))
        arr = np.ctypeslib.as_array(p, shape=(n.value,)).copy() if n.value else np.zeros(0, dtype=np.int32)
        w = _TABLE_WIDTH.get(name)
        return arr.reshape(-1, w) if w else arr

    def info(self, name: str) -> int:
        v = C.c_int64(0)
        _check(lib().fcp_plan_info(self.handle, INFO[name], C.byref(v)))
        return v.value

    def workspace_bytes(self, heads_per_pass=None):
        a, b, c = C.c_int64(0), C.c_int64(0), C.c_int64(0)
        _check(lib().fcp_plan_workspace_bytes(self.handle, int(heads_per_pass or self.hq), C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def bwd_scratch_bytes(self, kv_head_count=None) -> int:
        v = C.c_int64(0)
        _check(lib().fcp_plan_bwd_scratch_bytes(self.handle, int(kv_head_count or self.hkv), C.byref(v)))
        return v.value

    def host_workspace_bytes(self) -> int:
        v = C.c_int64(0)
        _check(lib().fcp_host_workspace_bytes(self.handle, C.byref(v)))
        return v.value

    def upload(self, stream=0):
        _check(lib().fcp_plan_upload(self.handle, C.c_void_p(stream)))
        return self

    def set_profiling(self, enable: bool):
        _check(lib().fcp_plan_set_profiling(self.handle, 1 if enable else 0))

    def kernel_ms(self, kind: int):
        n = C.c_int32(0)
        ms = C.c_float(0.0)
        _check(lib().fcp_plan_kernel_ms(self.handle, int(kind), C.byref(n), C.byref(ms)))
        return n.value, ms.value

    def device_status(self):
        st = np.zeros(4, dtype=np.int32)
        _check(lib().fcp_last_device_status(self.handle, st.ctypes.data_as(C.POINTER(C.c_int32))))
        return st


def fcp_plan_blocks(seqlens, cp_degrees, hq, hkv, head_dim, scale=0.0) -> Plan:
    return Plan(seqlens, cp_degrees, hq, hkv, head_dim, scale)


def fcp_plan_blocks_spans(seqlens, cp_degrees, spans, hq, hkv, head_dim, scale=0.0) -> Plan:
    return Plan(seqlens, cp_degrees, hq, hkv, head_dim, scale, spans=spans)


def fcp_span_mask_efficiency(length, spans) -> float:
    """eta_k of one sequence (Eq. 4): visible pairs over the causal count, minus 1."""
    flat = np.asarray([v for ab in spans for v in ab], dtype=np.int32)
    fl, flp = _i32(flat if flat.size else np.zeros(2, dtype=np.int32))
    eta = C.c_double(0.0)
    _check(lib().fcp_span_mask_efficiency(int(length), flp, len(spans), C.byref(eta)))
    return eta.value


def fcp_attn_fwd(plan: Plan, q, k, v, o_partial, lse_partial, head_begin=0, head_count=None, stream=0):
    hc = plan.hq - head_begin if head_count is None else head_count
    _check(lib().fcp_attn_fwd(plan.handle, _ptr(q), _ptr(k), _ptr(v), int(head_begin), int(hc), _ptr(o_partial),
                              _ptr(lse_partial), C.c_void_p(stream)))


def fcp_attn_fwd_merged(plan: Plan, q, k, v, o_partial, lse_partial, o, lse, head_begin=0, head_count=None, stream=0):
    hc = plan.hq - head_begin if head_count is None else head_count
    _check(lib().fcp_attn_fwd_merged(plan.handle, _ptr(q), _ptr(k), _ptr(v), int(head_begin), int(hc), _ptr(o_partial),
                                     _ptr(lse_partial), _ptr(o), _ptr(lse), C.c_void_p(stream)))


def fcp_attn_fwd_fused(plan: Plan, q, k, v, o, lse, head_begin=0, head_count=None, stream=0, o_f32=None):
    hc = plan.hq - head_begin if head_count is None else head_count
    _check(lib().fcp_attn_fwd_fused(plan.handle, _ptr(q), _ptr(k), _ptr(v), int(head_begin), int(hc), _ptr(o), _ptr(o_f32),
                                    _ptr(lse), C.c_void_p(stream)))


def fcp_lse_merge(plan: Plan, o_partial, lse_partial, o, lse, head_begin=0, head_count=None, stream=0, o_f32=None):
    hc = plan.hq - head_begin if head_count is None else head_count
    _check(lib().fcp_lse_merge(plan.handle, _ptr(o_partial), _ptr(lse_partial), int(head_begin), int(hc), _ptr(o),
                               _ptr(o_f32), _ptr(lse), C.c_void_p(stream)))


def fcp_attn_bwd(plan: Plan, q, k, v, o, d_o, lse, dq, dk, dv, scratch, scratch_bytes, stream=0):
    _check(lib().fcp_attn_bwd(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(dq), _ptr(dk),
                              _ptr(dv), _ptr(scratch), int(scratch_bytes), C.c_void_p(stream)))


def fcp_attn_bwd_heads(plan: Plan, q, k, v, o, d_o, lse, kv_head_begin, kv_head_count, dq, dk, dv, scratch, scratch_bytes,
                       stream=0):
    _check(lib().fcp_attn_bwd_heads(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), int(kv_head_begin),
                                    int(kv_head_count), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(scratch), int(scratch_bytes),
                                    C.c_void_p(stream)))


def fcp_attn_fwd_bwd_host(plan: Plan, q, k, v, d_o, o, lse, dq, dk, dv, workspace, workspace_bytes, stream=0):
    _check(lib().fcp_attn_fwd_bwd_host(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(d_o), _ptr(o), _ptr(lse), _ptr(dq),
                                       _ptr(dk), _ptr(dv), _ptr(workspace), int(workspace_bytes), C.c_void_p(stream)))


FCP_NOALLOC_MAX_BYTES = 32 << 20


def fcp_noalloc_bytes_needed(plan: Plan) -> int:
    v = C.c_int64(0)
    _check(lib().fcp_noalloc_bytes_needed(plan.handle, C.byref(v)))
    return v.value


def fcp_attn_bwd_noalloc(plan: Plan, q, k, v, o, d_o, lse, dq, dk, dv, stream=0):
    """Backward pass that allocates nothing: the plan need not be uploaded and no scratch is passed;
    the library's built-in arena (FCP_NOALLOC_MAX_BYTES per GPU) holds tables and scratch."""
    _check(lib().fcp_attn_bwd_noalloc(plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(d_o), _ptr(lse), _ptr(dq),
                                      _ptr(dk), _ptr(dv), C.c_void_p(stream)))


def fcp_noalloc_device_status():
    st = np.zeros(4, dtype=np.int32)
    _check(lib().fcp_noalloc_device_status(st.ctypes.data_as(C.POINTER(C.c_int32))))
    return st


def fcp_selftest_bounded_wait(limit_us=1000, stream=0):
    """Makes one bounded device-side wait run out on purpose (a barrier nobody arrives at, limit in
    microseconds) and returns the four status words it produced."""
    st = np.zeros(4, dtype=np.int32)
    _check(lib().fcp_selftest_bounded_wait(int(limit_us), st.ctypes.data_as(C.POINTER(C.c_int32)), C.c_void_p(stream)))
    return st
