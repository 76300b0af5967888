"""ctypes binding of include/et.h.  Function names and argument order follow the C ABI."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libet.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2312_14227_b200.build` "
        "(there is no fallback path)")
_lib = C.CDLL(LIB_PATH)

ET_OK = 0
ET_F32, ET_BF16 = 0, 1
ET_ACT_NONE, ET_ACT_GELU_TANH, ET_ACT_RELU = 0, 1, 2
ET_COST_STRICT, ET_COST_INCLUSIVE = 0, 1
ET_FLAG_FUSE_SGD = 1
ET_FLAG_DELTA_IS_SNAPSHOT = 2
ET_ERR_INVALID_ARG, ET_ERR_SHAPE, ET_ERR_DTYPE, ET_ERR_STATE = 1, 2, 3, 4
ET_ERR_WORKSPACE, ET_ERR_UNSUPPORTED, ET_ERR_CUDA, ET_ERR_TIMEOUT = 5, 6, 7, 8
ET_ERR_TOO_LARGE = 9
ET_ERR_GUARD = 10
ET_NOALLOC_SCRATCH_FLOATS = 1 << 20


class et_layer_desc(C.Structure):
    _fields_ = [("in_features", C.c_int32), ("out_features", C.c_int32), ("act", C.c_int32),
                ("fold", C.c_int32), ("residual_src", C.c_int32), ("kind", C.c_int32), ("eps", C.c_float),
                ("heads", C.c_int32), ("seq_len", C.c_int32), ("height", C.c_int32), ("width", C.c_int32),
                ("ksize", C.c_int32)]


ET_LAYER_DENSE, ET_LAYER_NORM, ET_LAYER_ATTENTION, ET_LAYER_IM2COL, ET_LAYER_BATCHNORM = 0, 1, 2, 3, 4


class et_optimizer_config(C.Structure):
    _fields_ = [("kind", C.c_int32), ("momentum", C.c_float), ("weight_decay", C.c_float),
                ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float)]


ET_OPT_SGD, ET_OPT_SGDW, ET_OPT_ADAM = 0, 1, 2


class et_dp_stats(C.Structure):
    _fields_ = [("table_full", C.c_int64), ("table_budget", C.c_int64), ("visited", C.c_int64),
                ("transitions", C.c_int64), ("rows_reached", C.c_int32), ("threads", C.c_int32)]

    def as_dict(self):
        return {k: int(getattr(self, k)) for k, _ in self._fields_}


class et_exec_report(C.Structure):
    _fields_ = [("dgrad", C.c_void_p), ("wgrad", C.c_void_p), ("bgrad", C.c_void_p), ("updated", C.c_void_p),
                ("deepest", C.c_int32), ("launches", C.c_int32), ("flops_executed", C.c_double)]


_vp, _i32, _i64, _u32, _f32, _f64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_float, C.c_double
_SIGS = {
    "et_stack_create": [_vp, _i32, _i64, _i32, C.POINTER(_vp)],
    "et_stack_destroy": [_vp],
    "et_stack_workspace_bytes": [_vp, C.POINTER(C.c_size_t)],
    "et_stack_set_option": [_vp, _i32, _i32],
    "et_stack_bind": [_vp, _vp, _vp, _vp, C.c_size_t, _vp],
    "et_stack_bind_master": [_vp, _vp, _vp],
    "et_forward_stack": [_vp, _vp, _vp, _vp],
    "et_loss_mse_grad": [_vp, _vp, _vp, _vp, _vp, _vp],
    "et_backward_elastic": [_vp, _vp, _vp, _i32, _vp, _vp, _vp, _u32, _f32, _vp, _vp],
    "et_backward_elastic_host": [_vp, _vp, _vp, _i32, _vp, _vp, _vp, _u32, _f32, _vp, _vp],
    "et_importance": [_vp, _vp, _i32, _vp, _vp, _vp, _vp],
    "et_tensor_metric": [_vp, _vp, _i32, _i32, _vp, _vp, _vp],
    "et_sgd_masked": [_vp, _vp, _i32, _vp, _f32, _vp],
    "et_update_masked": [_vp, _vp, _i32, _vp, _f32, _vp],
    "et_stack_set_optimizer": [_vp, _vp, _vp, _vp],
    "et_stack_set_optimizer_step": [_vp, _i32, _f32],
    "et_profile_costs": [_vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _vp],
    "et_time_selective": [_vp, _vp, _vp, _i32, _i32, _vp],
    "et_select_dp": [_vp, _vp, _vp, _i32, _f64, _f64, _i32, _i32, _vp, _vp, _vp],
    "et_select_dp_int": [_vp, _vp, _vp, _i32, _i64, _i32, _vp, _vp],
    "et_select_dp_ex": [_vp, _vp, _vp, _i32, _f64, _f64, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp],
    "et_select_dp_int_ex": [_vp, _vp, _vp, _i32, _i64, _i32, _i32, _i32, _vp, _vp, _vp],
    "et_device_status": [_vp, _vp],
    "et_debug_guard_regions": [_i32],
    "et_debug_check_guards": [_vp, _vp, _vp],
    "et_bias_grad_noalloc": [_vp, _i64, _i32, _i32, _vp, _vp],
    "et_timing_enable": [_vp, _i32],
    "et_timing_read": [_vp, _vp, _vp],
}
for _name, _args in _SIGS.items():
    _fn = getattr(_lib, _name)
    _fn.argtypes = _args
    _fn.restype = C.c_int
_lib.et_status_string.argtypes = [C.c_int]
_lib.et_status_string.restype = C.c_char_p
_lib.et_last_cuda_error.restype = C.c_int32
_lib.et_launch_count.restype = C.c_int64

EXPORTED_SYMBOLS = sorted(list(_SIGS) + ["et_status_string", "et_last_cuda_error", "et_launch_count"])


class EtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.et_status_string(status).decode()
        super().__init__(f"{where}: {msg} (status {status}, cuda error {_lib.et_last_cuda_error()})")


def _check(status: int, where: str):
    if status != ET_OK:
        raise EtError(status, where)


def et_status_string(status: int) -> str:
    return _lib.et_status_string(status).decode()


def et_launch_count() -> int:
    return int(_lib.et_launch_count())


def _ptr(t) -> Optional[int]:
    """Device / host pointer of a torch tensor, numpy array, int or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _ptr_array(seq: Optional[Sequence], n: int):
    if seq is None:
        return None
    assert len(seq) == n
    arr = (C.c_void_p * n)()
    for i, t in enumerate(seq):
        arr[i] = _ptr(t)
    return arr


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        return None
    return stream if isinstance(stream, int) else stream.cuda_stream


def _mask_arr(mask) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(mask, dtype=np.uint8))


# ---------------------------------------------------------------- host-only entry points
def et_time_selective(mask, t_dw, t_dy, variant: int = ET_COST_STRICT) -> float:
    m = _mask_arr(mask)
    w = np.ascontiguousarray(t_dw, dtype=np.float64)
    y = np.ascontiguousarray(t_dy, dtype=np.float64)
    out = C.c_double()
    _check(_lib.et_time_selective(_ptr(m), _ptr(w), _ptr(y), len(m), variant, C.addressof(out)), "et_time_selective")
    return out.value


def et_select_dp(importance, t_dw, t_dy, t_fwd: float, rho: float, Tq: int = 1000, variant: int = ET_COST_STRICT):
    I = np.ascontiguousarray(importance, dtype=np.float64)
    w = np.ascontiguousarray(t_dw, dtype=np.float64)
    y = np.ascontiguousarray(t_dy, dtype=np.float64)
    n = len(I)
    mask = np.zeros(max(n, 1), dtype=np.uint8)
    val, est = C.c_double(), C.c_double()
    _check(_lib.et_select_dp(_ptr(I), _ptr(w), _ptr(y), n, t_fwd, rho, Tq, variant, _ptr(mask),
                             C.addressof(val), C.addressof(est)), "et_select_dp")
    return mask[:n], val.value, est.value


def et_select_dp_ex(importance, t_dw, t_dy, t_fwd: float, rho: float, Tq: int = 1000, variant: int = ET_COST_STRICT,
                    threads: int = 1, prune: bool = True):
    """et_select_dp with the thread count and the pruning switch; also returns the run's et_dp_stats as a dict."""
    I = np.ascontiguousarray(importance, dtype=np.float64)
    w = np.ascontiguousarray(t_dw, dtype=np.float64)
    y = np.ascontiguousarray(t_dy, dtype=np.float64)
    n = len(I)
    mask = np.zeros(max(n, 1), dtype=np.uint8)
    val, est = C.c_double(), C.c_double()
    st = et_dp_stats()
    _check(_lib.et_select_dp_ex(_ptr(I), _ptr(w), _ptr(y), n, t_fwd, rho, Tq, variant, threads, 1 if prune else 0,
                                _ptr(mask), C.addressof(val), C.addressof(est), C.addressof(st)), "et_select_dp_ex")
    return mask[:n], val.value, est.value, st.as_dict()


def et_select_dp_int_ex(importance, t_dw, t_dy, budget: int, variant: int = ET_COST_STRICT, threads: int = 1,
                        prune: bool = True):
    I = np.ascontiguousarray(importance, dtype=np.float64)
    w = np.ascontiguousarray(t_dw, dtype=np.int64)
    y = np.ascontiguousarray(t_dy, dtype=np.int64)
    n = len(I)
    mask = np.zeros(max(n, 1), dtype=np.uint8)
    val = C.c_double()
    st = et_dp_stats()
    _check(_lib.et_select_dp_int_ex(_ptr(I), _ptr(w), _ptr(y), n, int(budget), variant, threads, 1 if prune else 0,
                                    _ptr(mask), C.addressof(val), C.addressof(st)), "et_select_dp_int_ex")
    return mask[:n], val.value, st.as_dict()


def et_select_dp_int(importance, t_dw, t_dy, budget: int, variant: int = ET_COST_STRICT):
    I = np.ascontiguousarray(importance, dtype=np.float64)
    w = np.ascontiguousarray(t_dw, dtype=np.int64)
    y = np.ascontiguousarray(t_dy, dtype=np.int64)
    n = len(I)
    mask = np.zeros(max(n, 1), dtype=np.uint8)
    val = C.c_double()
    _check(_lib.et_select_dp_int(_ptr(I), _ptr(w), _ptr(y), n, int(budget), variant, _ptr(mask),
                                 C.addressof(val)), "et_select_dp_int")
    return mask[:n], val.value


# ---------------------------------------------------------------- stack object
class Report:
    """Host copy of et_exec_report."""

    def __init__(self, L: int):
        self.dgrad = np.zeros(L, dtype=np.uint8)
        self.wgrad = np.zeros(L, dtype=np.uint8)
        self.bgrad = np.zeros(L, dtype=np.uint8)
        self.updated = np.zeros(2 * L, dtype=np.uint8)
        self.c = et_exec_report(_ptr(self.dgrad), _ptr(self.wgrad), _ptr(self.bgrad), _ptr(self.updated), 0, 0, 0.0)

    deepest = property(lambda self: self.c.deepest)
    launches = property(lambda self: self.c.launches)
    flops_executed = property(lambda self: self.c.flops_executed)


class Stack:
    """Owns the opaque et_stack handle.  Layers: sequence of objects / tuples with
    in_features, out_features, act, fold, residual_src."""

    def __init__(self, layers, M: int, dtype: int):
        self.L = len(layers)
        self.M = int(M)
        self.dtype = dtype
        descs = (et_layer_desc * max(self.L, 1))()
        for i, ly in enumerate(layers):
            if isinstance(ly, (tuple, list)):
                descs[i] = et_layer_desc(*ly)
            else:
                descs[i] = et_layer_desc(ly.in_features, ly.out_features, ly.act, ly.fold, ly.residual_src,
                                         getattr(ly, "kind", ET_LAYER_DENSE), getattr(ly, "eps", 0.0),
                                         getattr(ly, "heads", 0), getattr(ly, "seq", 0), getattr(ly, "height", 0),
                                         getattr(ly, "width", 0), getattr(ly, "ksize", 0))
        self.out_width = (descs[self.L - 1].out_features // max(descs[self.L - 1].fold, 1)) if self.L else 0
        h = C.c_void_p()
        _check(_lib.et_stack_create(descs, self.L, self.M, dtype, C.byref(h)), "et_stack_create")
        self.handle = h
        self._keep = []

    def close(self):
        if getattr(self, "handle", None):
            _lib.et_stack_destroy(self.handle)
            self.handle = None

    __del__ = close


def et_stack_create(layers, M: int, dtype: int) -> Stack:
    return Stack(layers, M, dtype)


def et_stack_destroy(s: Stack):
    s.close()


ET_OPTION_TWO_STREAMS, ET_OPTION_LAUNCH_OVERLAP, ET_OPTION_TILE_PLAN, ET_OPTION_GEMM_LIST = 1, 2, 3, 4
ET_OPTION_LIST_COOPERATIVE = 5
ET_TILE_PLAN_AUTO, ET_TILE_PLAN_ALONE, ET_TILE_PLAN_SHARED = 0, 1, 2


def et_stack_set_option(s: Stack, option: int, value: int):
    _check(_lib.et_stack_set_option(s.handle, int(option), int(value)), "et_stack_set_option")


def et_stack_workspace_bytes(s: Stack) -> int:
    out = C.c_size_t()
    _check(_lib.et_stack_workspace_bytes(s.handle, C.byref(out)), "et_stack_workspace_bytes")
    return out.value


def et_stack_bind(s: Stack, W, b, workspace, workspace_bytes: Optional[int] = None, stream=None):
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    s._keep = [list(W), list(b), workspace]          # keep the tensors alive while bound
    _check(_lib.et_stack_bind(s.handle, _ptr_array(W, s.L), _ptr_array(b, s.L), _ptr(workspace),
                              workspace_bytes, _stream_ptr(stream)), "et_stack_bind")


def et_stack_bind_master(s: Stack, W32, b32):
    s._keep_master = [list(W32), list(b32)] if W32 is not None else None
    _check(_lib.et_stack_bind_master(s.handle, _ptr_array(W32, s.L) if W32 is not None else None,
                                     _ptr_array(b32, s.L) if b32 is not None else None), "et_stack_bind_master")


def et_forward_stack(s: Stack, x, y, stream=None):
    _check(_lib.et_forward_stack(s.handle, _ptr(x), _ptr(y), _stream_ptr(stream)), "et_forward_stack")


def et_loss_mse_grad(s: Stack, y, target, dY, loss_dev=None, stream=None):
    _check(_lib.et_loss_mse_grad(s.handle, _ptr(y), _ptr(target), _ptr(dY), _ptr(loss_dev),
                                 _stream_ptr(stream)), "et_loss_mse_grad")


def _backward(fn, name, s, dY, mask, grads, delta, importance, flags, lr, report, stream):
    m = _mask_arr(mask)
    n = len(m)
    _check(fn(s.handle, _ptr(dY), _ptr(m), n,
              _ptr_array(grads, n) if grads is not None else None,
              _ptr_array(delta, n) if delta is not None else None,
              _ptr(importance), flags, lr,
              C.addressof(report.c) if report is not None else None, _stream_ptr(stream)), name)


def et_backward_elastic(s: Stack, dY, mask, grads=None, delta=None, importance_dev=None, flags: int = 0,
                        lr: float = 0.0, report: Optional[Report] = None, stream=None):
    _backward(_lib.et_backward_elastic, "et_backward_elastic", s, dY, mask, grads, delta, importance_dev,
              flags, lr, report, stream)


def et_backward_elastic_host(s: Stack, dY_host, mask, grads=None, delta=None, importance_host=None,
                             flags: int = 0, lr: float = 0.0, report: Optional[Report] = None, stream=None):
    _backward(_lib.et_backward_elastic_host, "et_backward_elastic_host", s, dY_host, mask, grads, delta,
              importance_host, flags, lr, report, stream)


def et_importance(s: Stack, mask, grads, delta, importance_dev, stream=None):
    m = _mask_arr(mask)
    _check(_lib.et_importance(s.handle, _ptr(m), len(m), _ptr_array(grads, len(m)), _ptr_array(delta, len(m)),
                              _ptr(importance_dev), _stream_ptr(stream)), "et_importance")


ET_METRIC_WEIGHT_MAGNITUDE, ET_METRIC_GRADIENT_MAGNITUDE = 1, 2


def et_tensor_metric(s: Stack, mask, kind: int, grads, metric_dev, stream=None):
    m = _mask_arr(mask)
    g = _ptr_array(grads, len(m)) if grads is not None else None
    _check(_lib.et_tensor_metric(s.handle, _ptr(m), len(m), kind, g, _ptr(metric_dev), _stream_ptr(stream)),
           "et_tensor_metric")


def et_sgd_masked(s: Stack, mask, grads, lr: float, stream=None):
    m = _mask_arr(mask)
    _check(_lib.et_sgd_masked(s.handle, _ptr(m), len(m), _ptr_array(grads, len(m)), lr, _stream_ptr(stream)),
           "et_sgd_masked")


def et_update_masked(s: Stack, mask, grads, lr: float, stream=None):
    m = _mask_arr(mask)
    _check(_lib.et_update_masked(s.handle, _ptr(m), len(m), _ptr_array(grads, len(m)), lr, _stream_ptr(stream)),
           "et_update_masked")


def et_stack_set_optimizer(s: Stack, kind: int, state1=None, state2=None, momentum=0.9, weight_decay=0.0,
                           beta1=0.9, beta2=0.999, eps=1e-8):
    cfg = et_optimizer_config(kind, momentum, weight_decay, beta1, beta2, eps)
    s._keep_opt = [state1, state2]
    n = 2 * s.L
    _check(_lib.et_stack_set_optimizer(s.handle, C.addressof(cfg),
                                       _ptr_array(state1, n) if state1 is not None else None,
                                       _ptr_array(state2, n) if state2 is not None else None), "et_stack_set_optimizer")


def et_stack_set_optimizer_step(s: Stack, step: int, weight_decay: float = 0.0):
    _check(_lib.et_stack_set_optimizer_step(s.handle, int(step), float(weight_decay)), "et_stack_set_optimizer_step")


def et_profile_costs(s: Stack, x, y, dY, iters: int = 20, stream=None):
    t_dw = np.zeros(2 * s.L)
    t_dy = np.zeros(2 * s.L)
    t_fwd = C.c_double()
    _check(_lib.et_profile_costs(s.handle, _ptr(x), _ptr(y), _ptr(dY), iters, _ptr(t_dw), _ptr(t_dy),
                                 C.addressof(t_fwd), _stream_ptr(stream)), "et_profile_costs")
    return t_dw, t_dy, t_fwd.value


KERNEL_CLASSES = ("forward", "dgrad", "wgrad", "wgrad_reduce", "bgrad", "other", "norm", "attention", "gemm_list")


def et_timing_enable(s: Stack, on: bool):
    _check(_lib.et_timing_enable(s.handle, 1 if on else 0), "et_timing_enable")


def et_timing_read(s: Stack):
    """{class name: (milliseconds, launches)} since the last read."""
    ms = np.zeros(len(KERNEL_CLASSES), dtype=np.float64)
    n = np.zeros(len(KERNEL_CLASSES), dtype=np.int64)
    _check(_lib.et_timing_read(s.handle, _ptr(ms), _ptr(n)), "et_timing_read")
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_CLASSES)}


def et_bias_grad_noalloc(dZ, M: int, width: int, dtype: int, db, stream=None):
    """Column sums of dZ [M x width] into db (float32[width]) using the library's built-in
    scratch instead of a workspace: for callers that are not allowed to allocate device
    memory.  Problems over ET_NOALLOC_SCRATCH_FLOATS raise EtError(ET_ERR_TOO_LARGE)."""
    _check(_lib.et_bias_grad_noalloc(_ptr(dZ), int(M), int(width), dtype, _ptr(db), _stream_ptr(stream)),
           "et_bias_grad_noalloc")


def et_debug_guard_regions(on: bool):
    _check(_lib.et_debug_guard_regions(1 if on else 0), "et_debug_guard_regions")


def et_debug_check_guards(s: Stack, stream=None):
    """(status, index of the first damaged region or -1)."""
    bad = C.c_int32(-1)
    st = int(_lib.et_debug_check_guards(s.handle, _stream_ptr(stream), C.addressof(bad)))
    return st, bad.value


def et_device_status(s: Stack, stream=None) -> int:
    return int(_lib.et_device_status(s.handle, _stream_ptr(stream)))


__all__ = [n for n in dir() if n.startswith(("et_", "ET_"))] + ["Stack", "Report", "EtError", "LIB_PATH",
                                                                 "EXPORTED_SYMBOLS", "KERNEL_CLASSES"]
