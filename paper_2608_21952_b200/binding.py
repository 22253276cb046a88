"""Thin ctypes binding of libssdi8 (argument marshalling only).

The functions carry the names of the C entry points declared in include/ssdi8.h
and take torch CUDA tensors; every step of the computation runs inside the
library's kernels.  There is no fallback: if the library cannot be loaded the
import raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

_LIB_PATH = _build.LIB
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2608_21952_b200.build` "
        "(nvcc, sm_100a); there is no CPU or PyTorch fallback")
_lib = C.CDLL(_LIB_PATH)

OK = 0
ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_UNSUPPORTED = \
    -1, -2, -3, -4, -5, -6, -7, -8

FLAG_FP16_OPERAND = 1 << 0
FLAG_INT8_STATE = 1 << 1
FLAG_Y_FP16, FLAG_Y_BF16 = 1 << 2, 1 << 3
FLAG_DT_SOFTPLUS = 1 << 4
PHASE_CUMSUM, PHASE_BMM, PHASE_CHUNK_STATE, PHASE_STATE_PASSING, PHASE_SCAN = (1 << k for k in range(8, 13))

EXPORTS = ("ssdi8_status_string", "ssdi8_workspace_bytes", "ssdi8_quantize_act",
           "ssdi8_chunk_scan_fwd", "ssdi8_chunk_scan_fwd_static", "ssdi8_calibrate",
           "ssdi8_state_passing", "ssdi8_ssd_step", "ssdi8_mean_correction",
           "ssdi8_mean_correction_workspace_bytes", "ssdi8_quantize_entry",
           "ssdi8_layer_fwd", "ssdi8_layer_fwd_workspace_bytes",
           "ssdi8_layer_fwd_host", "ssdi8_layer_fwd_host_scratch_bytes",
           "ssdi8_int8_mma_peak", "ssdi8_selftest_bounded_wait", "ssdi8_softplus_dt")
STATIC_WORKSPACE_BYTES = 16 << 20


class Dims(C.Structure):
    _fields_ = [(k, C.c_int32) for k in
                ("batch", "seqlen", "nheads", "headdim", "dstate", "ngroups", "chunk")]


_FWD_FIELDS = ("xq", "Bq", "Cq", "s_x", "s_B", "s_C", "dt", "A", "D", "corr", "s_xs", "s_cb", "s_h",
               "init_state", "y", "final_state", "status",
               "tap_cs", "tap_acc_cb", "tap_CBq", "tap_Xsq", "tap_acc_st", "tap_loc", "tap_prev",
               "tap_hq", "tap_acc_off", "tap_rowmax", "tap_Mq", "tap_acc_diag", "dt_bias")


class FwdArgs(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in _FWD_FIELDS]


_LAYER_FIELDS = ("x", "B", "C", "dt", "A", "D", "corr", "s_x", "s_B", "s_C", "s_xs", "s_cb", "s_h",
                "init_state", "y", "final_state", "status")


_HOST_SIDE = ("x", "B", "C", "dt", "y", "final_state", "status")


class LayerArgs(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in _LAYER_FIELDS]


_lib.ssdi8_status_string.restype = C.c_char_p
_lib.ssdi8_status_string.argtypes = [C.c_int32]
_lib.ssdi8_workspace_bytes.restype = C.c_size_t
_lib.ssdi8_workspace_bytes.argtypes = [C.POINTER(Dims), C.c_uint32]
_lib.ssdi8_quantize_act.restype = C.c_int32
_lib.ssdi8_quantize_act.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p,
                                    C.c_int32, C.c_void_p, C.c_void_p]
_lib.ssdi8_chunk_scan_fwd.restype = C.c_int32
_lib.ssdi8_chunk_scan_fwd.argtypes = [C.POINTER(Dims), C.POINTER(FwdArgs), C.c_uint32, C.c_void_p,
                                      C.c_size_t, C.c_void_p]
_lib.ssdi8_chunk_scan_fwd_static.restype = C.c_int32
_lib.ssdi8_chunk_scan_fwd_static.argtypes = [C.POINTER(Dims), C.POINTER(FwdArgs), C.c_uint32, C.c_void_p]
_lib.ssdi8_calibrate.restype = C.c_int32
_lib.ssdi8_calibrate.argtypes = [C.POINTER(Dims), C.POINTER(FwdArgs), C.c_void_p, C.c_void_p,
                                 C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
_lib.ssdi8_mean_correction_workspace_bytes.restype = C.c_size_t
_lib.ssdi8_mean_correction_workspace_bytes.argtypes = [C.c_int64]
_lib.ssdi8_mean_correction.restype = C.c_int32
_lib.ssdi8_mean_correction.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_float, C.c_void_p,
                                       C.c_void_p, C.c_size_t, C.c_void_p]
_lib.ssdi8_quantize_entry.restype = C.c_int32
_lib.ssdi8_quantize_entry.argtypes = [C.c_void_p, C.c_int32, C.c_int64, C.c_int32, C.c_int32, C.c_int32] + \
    [C.c_void_p] * 7
_lib.ssdi8_state_passing.restype = C.c_int32
_lib.ssdi8_state_passing.argtypes = [C.POINTER(Dims)] + [C.c_void_p] * 8
_lib.ssdi8_ssd_step.restype = C.c_int32
_lib.ssdi8_ssd_step.argtypes = [C.POINTER(Dims)] + [C.c_void_p] * 13


class SSDi8Error(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {ssdi8_status_string(code)} ({code})")


def _check(code: int, where: str) -> None:
    if code != OK:
        raise SSDi8Error(code, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def dims_of(cfg) -> Dims:
    return Dims(cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim, cfg.dstate, cfg.ngroups, cfg.chunk)


def ssdi8_status_string(code: int) -> str:
    return _lib.ssdi8_status_string(int(code)).decode()


def ssdi8_workspace_bytes(dims: Dims, flags: int = 0) -> int:
    return int(_lib.ssdi8_workspace_bytes(C.byref(dims), flags))


def ssdi8_quantize_act(inp, R: int, Ch: int, I: int, scale, mode: int, out, stream=None) -> None:
    _check(_lib.ssdi8_quantize_act(_ptr(inp), R, Ch, I, _ptr(scale), mode, _ptr(out), _stream(stream)),
           "ssdi8_quantize_act")


def make_fwd_args(**tensors) -> FwdArgs:
    a = FwdArgs()
    for k, v in tensors.items():
        if k not in _FWD_FIELDS:
            raise KeyError(k)
        setattr(a, k, _ptr(v))
    a._keepalive = dict(tensors)  # the struct holds raw pointers: keep the tensors alive with it
    return a


def ssdi8_chunk_scan_fwd(dims: Dims, args: FwdArgs, workspace, flags: int = 0, stream=None) -> None:
    _check(_lib.ssdi8_chunk_scan_fwd(C.byref(dims), C.byref(args), flags, _ptr(workspace),
                                     workspace.numel() * workspace.element_size(), _stream(stream)),
           "ssdi8_chunk_scan_fwd")


def ssdi8_chunk_scan_fwd_static(dims: Dims, args: FwdArgs, flags: int = 0, stream=None) -> None:
    """Forward pass on the library's built-in scratch: no workspace argument, no allocation.
    For callers that cannot allocate device memory; raises SSDi8Error(ERR_WORKSPACE) when the
    dimensions need more than STATIC_WORKSPACE_BYTES."""
    _check(_lib.ssdi8_chunk_scan_fwd_static(C.byref(dims), C.byref(args), flags, _stream(stream)),
           "ssdi8_chunk_scan_fwd_static")


def ssdi8_calibrate(dims: Dims, args: FwdArgs, s_xs, s_cb, s_h, workspace, stream=None) -> None:
    _check(_lib.ssdi8_calibrate(C.byref(dims), C.byref(args), _ptr(s_xs), _ptr(s_cb), _ptr(s_h),
                                _ptr(workspace), workspace.numel() * workspace.element_size(),
                                _stream(stream)), "ssdi8_calibrate")


_lib.ssdi8_layer_fwd_host_scratch_bytes.restype = C.c_size_t
_lib.ssdi8_layer_fwd_host_scratch_bytes.argtypes = [C.POINTER(Dims), C.c_uint32]
_lib.ssdi8_layer_fwd_workspace_bytes.restype = C.c_size_t
_lib.ssdi8_layer_fwd_workspace_bytes.argtypes = [C.POINTER(Dims), C.c_uint32]
_lib.ssdi8_layer_fwd.restype = C.c_int32
_lib.ssdi8_layer_fwd.argtypes = [C.POINTER(Dims), C.POINTER(LayerArgs), C.c_void_p, C.c_size_t, C.c_uint32,
                                 C.c_void_p]
_lib.ssdi8_layer_fwd_host.restype = C.c_int32
_lib.ssdi8_layer_fwd_host.argtypes = [C.POINTER(Dims), C.POINTER(LayerArgs), C.c_void_p, C.c_size_t, C.c_uint32,
                                      C.c_void_p]


def make_layer_args(host: bool = False, **tensors) -> LayerArgs:
    """Arguments of ssdi8_layer_fwd (host=False: all device tensors) or ssdi8_layer_fwd_host
    (host=True: x, B, C, dt, y, final_state, status are host tensors, pinned; the rest device tensors)."""
    a = LayerArgs()
    for k, v in tensors.items():
        if k not in _LAYER_FIELDS:
            raise KeyError(k)
        if host and k in _HOST_SIDE and v is not None:
            assert not v.is_cuda and v.is_contiguous(), f"{k} must be a contiguous host tensor"
            setattr(a, k, v.data_ptr())
        else:
            setattr(a, k, _ptr(v))
    a._keepalive = dict(tensors)
    return a


def make_host_args(**tensors) -> LayerArgs:
    return make_layer_args(host=True, **tensors)


def ssdi8_layer_fwd_workspace_bytes(dims: Dims, flags: int = 0) -> int:
    return int(_lib.ssdi8_layer_fwd_workspace_bytes(C.byref(dims), flags))


def ssdi8_layer_fwd(dims: Dims, args: LayerArgs, workspace, flags: int = 0, stream=None) -> None:
    _check(_lib.ssdi8_layer_fwd(C.byref(dims), C.byref(args), _ptr(workspace),
                                workspace.numel() * workspace.element_size(), flags, _stream(stream)),
           "ssdi8_layer_fwd")


def ssdi8_layer_fwd_host_scratch_bytes(dims: Dims, flags: int = 0) -> int:
    return int(_lib.ssdi8_layer_fwd_host_scratch_bytes(C.byref(dims), flags))


def ssdi8_layer_fwd_host(dims: Dims, args: LayerArgs, scratch, flags: int = 0, stream=None) -> None:
    _check(_lib.ssdi8_layer_fwd_host(C.byref(dims), C.byref(args), _ptr(scratch),
                                     scratch.numel() * scratch.element_size(), flags, _stream(stream)),
           "ssdi8_layer_fwd_host")


_ENTRY_DTYPES = {torch.float32: 0, torch.float16: 1, torch.bfloat16: 2}


def ssdi8_quantize_entry(xBC, T: int, D: int, G: int, N: int, s_x, s_B, s_C, xq, Bq, Cq, stream=None) -> None:
    _check(_lib.ssdi8_quantize_entry(_ptr(xBC), _ENTRY_DTYPES[xBC.dtype], T, D, G, N, _ptr(s_x), _ptr(s_B),
                                     _ptr(s_C), _ptr(xq), _ptr(Bq), _ptr(Cq), _stream(stream)),
           "ssdi8_quantize_entry")


def ssdi8_mean_correction_workspace_bytes(Ch: int) -> int:
    return int(_lib.ssdi8_mean_correction_workspace_bytes(Ch))


def ssdi8_mean_correction(y_ref, y_q, R: int, Ch: int, eta: float, corr, workspace, stream=None) -> None:
    _check(_lib.ssdi8_mean_correction(_ptr(y_ref), _ptr(y_q), R, Ch, eta, _ptr(corr), _ptr(workspace),
                                      workspace.numel() * workspace.element_size(), _stream(stream)),
           "ssdi8_mean_correction")


def ssdi8_state_passing(dims: Dims, loc, gamma, init_state, prev, final_state, hq, s_h,
                        stream=None) -> None:
    _check(_lib.ssdi8_state_passing(C.byref(dims), _ptr(loc), _ptr(gamma), _ptr(init_state), _ptr(prev),
                                    _ptr(final_state), _ptr(hq), _ptr(s_h), _stream(stream)),
           "ssdi8_state_passing")


def ssdi8_ssd_step(dims: Dims, xq, s_x, Bq, s_B, Cq, s_C, dt, A, D, corr, state, y, stream=None) -> None:
    _check(_lib.ssdi8_ssd_step(C.byref(dims), _ptr(xq), _ptr(s_x), _ptr(Bq), _ptr(s_B), _ptr(Cq),
                               _ptr(s_C), _ptr(dt), _ptr(A), _ptr(D), _ptr(corr), _ptr(state), _ptr(y),
                               _stream(stream)), "ssdi8_ssd_step")


_lib.ssdi8_int8_mma_peak.restype = C.c_int32
_lib.ssdi8_int8_mma_peak.argtypes = [C.c_int64, C.POINTER(C.c_double), C.c_void_p, C.c_void_p]
_lib.ssdi8_selftest_bounded_wait.restype = C.c_int32
_lib.ssdi8_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_void_p]


_lib.ssdi8_softplus_dt.restype = C.c_int32
_lib.ssdi8_softplus_dt.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p]


def ssdi8_softplus_dt(dt_raw, dt_bias, rows: int, H: int, dt, stream=None) -> None:
    _check(_lib.ssdi8_softplus_dt(_ptr(dt_raw), _ptr(dt_bias), rows, H, _ptr(dt), _stream(stream)),
           "ssdi8_softplus_dt")


def ssdi8_int8_mma_peak(mma_per_sm: int, status=None, stream=None) -> float:
    """Launches the dense INT8 MMA loop; returns the number of integer operations of the launch."""
    ops = C.c_double(0.0)
    _check(_lib.ssdi8_int8_mma_peak(mma_per_sm, C.byref(ops), _ptr(status), _stream(stream)),
           "ssdi8_int8_mma_peak")
    return float(ops.value)


def ssdi8_selftest_bounded_wait(status, stream=None) -> None:
    _check(_lib.ssdi8_selftest_bounded_wait(_ptr(status), _stream(stream)), "ssdi8_selftest_bounded_wait")


def alloc_workspace(dims: Dims, device="cuda", flags: int = 0):
    n = ssdi8_workspace_bytes(dims, flags)
    if n == 0:
        raise SSDi8Error(ERR_SHAPE, "ssdi8_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)
