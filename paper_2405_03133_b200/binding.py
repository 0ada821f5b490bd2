"""ctypes binding of liblory.so: same names as include/lory.h, argument marshalling only.

Tensors are torch CUDA tensors (torch supplies device memory and streams); every
step of the layer runs inside the library's kernels.  There is no fallback: if the
library is missing or the device is not a B200-class GPU, calls raise.
"""
from __future__ import annotations

import ctypes
import os

LORY_FP32 = 0
LORY_BF16 = 1
LORY_FLAG_SIMT = 1
LORY_FLAG_REUSE_MERGED = 2
LORY_FLAG_PREFIX_ROUTING = 4
LORY_FLAG_FIRST_SEGMENT_GRAD = 8
LORY_FLAG_ACCUMULATE_GRADS = 16
LORY_FLAG_CHUNKED_ADJOINT = 32

_HERE = os.path.dirname(os.path.abspath(__file__))
# LORY_LIBRARY selects another build of the same ABI, e.g. the bounds-checking liblory_debug.so
LIB_PATH = os.environ.get("LORY_LIBRARY") or os.path.join(_HERE, "liblory.so")


class LoryError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(text)
        self.status = status


class lory_dims(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int), ("L", ctypes.c_int), ("T", ctypes.c_int), ("d", ctypes.c_int),
                ("f", ctypes.c_int), ("E", ctypes.c_int), ("dtype", ctypes.c_int), ("flags", ctypes.c_int)]

    @property
    def S(self):
        return self.B * (self.L // self.T)


_lib = None
_vp, _sz = ctypes.c_void_p, ctypes.c_size_t
_DP = ctypes.POINTER(lory_dims)
_SIGNATURES = {
    "lory_status_string": (ctypes.c_char_p, [ctypes.c_int]),
    "lory_last_cuda_error": (ctypes.c_char_p, []),
    "lory_last_launch_count": (ctypes.c_int, []),
    "lory_moe_workspace_bytes": (ctypes.c_int, [_DP, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "lory_moe_forward": (ctypes.c_int, [_DP] + [_vp] * 9 + [_sz, _vp]),
    "lory_moe_ffn": (ctypes.c_int, [_DP] + [_vp] * 7 + [_sz, _vp]),
    "lory_moe_backward": (ctypes.c_int, [_DP] + [_vp] * 13 + [_sz, _vp]),
    "lory_moe_step_host_bytes": (ctypes.c_int, [_DP, ctypes.POINTER(_sz)]),
    "lory_moe_step_host": (ctypes.c_int, [_DP] + [_vp] * 14 + [_sz, _vp]),
    "lory_block_workspace_bytes": (ctypes.c_int, [_DP, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]),
    "lory_block_forward": (ctypes.c_int, [_DP, _vp, _vp, ctypes.c_float] + [_vp] * 8 + [_sz, _vp]),
    "lory_block_backward": (ctypes.c_int, [_DP] + [_vp] * 15 + [_sz, _vp]),
    "lory_moe_step_host_pipeline_bytes": (ctypes.c_int, [_DP, ctypes.POINTER(_sz)]),
    "lory_moe_step_host_enqueue": (ctypes.c_int, [_DP, ctypes.c_int] + [_vp] * 14 + [_sz, _vp]),
    "lory_moe_step_host_wait": (ctypes.c_int, [ctypes.c_int]),
    "lory_check_status": (ctypes.c_int, [_DP, _vp, _sz, _vp]),
    "lory_route_noalloc": (ctypes.c_int, [_DP] + [_vp] * 5),
    "lory_expert_utilization": (ctypes.c_int, [_vp, ctypes.c_int, ctypes.c_int, _vp, _vp]),
    "lory_selftest_bounded_wait": (ctypes.c_int, [_DP, _vp, _sz, _vp]),
    "lory_debug_build": (ctypes.c_int, []),
    "lory_selftest_debug_bounds": (ctypes.c_int, [_DP, _vp, _sz, _vp]),
    "lory_probe_l2_ring": (ctypes.c_int, [_vp, _sz, _sz] + [ctypes.c_int] * 5 + [ctypes.POINTER(ctypes.c_float), _vp]),
    "lory_profile_enable": (ctypes.c_int, [ctypes.c_int]),
    "lory_profile_read": (ctypes.c_int, [ctypes.c_int, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_float)]),
}


def load():
    """Loads liblory.so (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise LoryError(-100, f"{LIB_PATH} not found: build it with `python -m paper_2405_03133_b200.build`")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def exported_symbols():
    return list(_SIGNATURES)


def _check(status):
    if status != 0:
        lib = load()
        text = lib.lory_status_string(status).decode()
        if status == -6:
            text += " -- " + lib.lory_last_cuda_error().decode()
        raise LoryError(status, text)


def _ptr(t):
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        if not t.is_contiguous():
            raise ValueError("tensors passed to the Lory library must be contiguous")
        return ctypes.c_void_p(t.data_ptr())
    return ctypes.c_void_p(int(t))


def _nbytes(t):
    return t.numel() * t.element_size()


def _stream(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(getattr(stream, "cuda_stream", stream))


def make_dims(B, L, T, d, f, E, dtype, flags=0):
    if isinstance(dtype, str):
        dtype = {"fp32": LORY_FP32, "bf16": LORY_BF16}[dtype]
    return lory_dims(B, L, T, d, f, E, dtype, flags)


def lory_status_string(status):
    return load().lory_status_string(status).decode()


def lory_last_launch_count():
    return load().lory_last_launch_count()


def lory_moe_workspace_bytes(dims):
    fwd, bwd = _sz(0), _sz(0)
    _check(load().lory_moe_workspace_bytes(ctypes.byref(dims), ctypes.byref(fwd), ctypes.byref(bwd)))
    return fwd.value, bwd.value


def lory_moe_forward(dims, x, w_r, w1, w2, w3, y, route_w, route_p, workspace, stream=None):
    _check(load().lory_moe_forward(ctypes.byref(dims), _ptr(x), _ptr(w_r), _ptr(w1), _ptr(w2), _ptr(w3), _ptr(y),
                                   _ptr(route_w), _ptr(route_p), _ptr(workspace), _nbytes(workspace),
                                   _stream(stream)))


def lory_moe_ffn(dims, x, route_w, w1, w2, w3, y, workspace, stream=None):
    _check(load().lory_moe_ffn(ctypes.byref(dims), _ptr(x), _ptr(route_w), _ptr(w1), _ptr(w2), _ptr(w3), _ptr(y),
                               _ptr(workspace), _nbytes(workspace), _stream(stream)))


def lory_moe_backward(dims, x, w_r, w1, w2, w3, dy, dx, dw_r, dw1, dw2, dw3, d_route_w, workspace, stream=None):
    _check(load().lory_moe_backward(ctypes.byref(dims), _ptr(x), _ptr(w_r), _ptr(w1), _ptr(w2), _ptr(w3), _ptr(dy),
                                    _ptr(dx), _ptr(dw_r), _ptr(dw1), _ptr(dw2), _ptr(dw3), _ptr(d_route_w),
                                    _ptr(workspace), _nbytes(workspace), _stream(stream)))


def lory_moe_step_host_bytes(dims):
    n = _sz(0)
    _check(load().lory_moe_step_host_bytes(ctypes.byref(dims), ctypes.byref(n)))
    return n.value


def lory_moe_step_host(dims, x_host, dy_host, w_r, w1, w2, w3, y_host, dx_host, route_w_host, dw_r, dw1, dw2, dw3,
                       arena, stream=None):
    _check(load().lory_moe_step_host(ctypes.byref(dims), _ptr(x_host), _ptr(dy_host), _ptr(w_r), _ptr(w1), _ptr(w2),
                                     _ptr(w3), _ptr(y_host), _ptr(dx_host), _ptr(route_w_host), _ptr(dw_r),
                                     _ptr(dw1), _ptr(dw2), _ptr(dw3), _ptr(arena), _nbytes(arena),
                                     _stream(stream)))


def lory_block_workspace_bytes(dims):
    f, b = _sz(0), _sz(0)
    _check(load().lory_block_workspace_bytes(ctypes.byref(dims), ctypes.byref(f), ctypes.byref(b)))
    return f.value, b.value


def lory_block_forward(dims, x, gamma, eps, w_r, w1, w2, w3, y, route_w, route_p, workspace, stream=None):
    _check(load().lory_block_forward(ctypes.byref(dims), _ptr(x), _ptr(gamma), ctypes.c_float(eps), _ptr(w_r), _ptr(w1),
                                     _ptr(w2), _ptr(w3), _ptr(y), _ptr(route_w), _ptr(route_p), _ptr(workspace),
                                     _nbytes(workspace), _stream(stream)))


def lory_block_backward(dims, x, gamma, w_r, w1, w2, w3, dy, dx, dgamma, dw_r, dw1, dw2, dw3, d_route_w, workspace,
                        stream=None):
    _check(load().lory_block_backward(ctypes.byref(dims), _ptr(x), _ptr(gamma), _ptr(w_r), _ptr(w1), _ptr(w2), _ptr(w3),
                                      _ptr(dy), _ptr(dx), _ptr(dgamma), _ptr(dw_r), _ptr(dw1), _ptr(dw2), _ptr(dw3),
                                      _ptr(d_route_w), _ptr(workspace), _nbytes(workspace), _stream(stream)))


def lory_moe_step_host_pipeline_bytes(dims):
    n = _sz(0)
    _check(load().lory_moe_step_host_pipeline_bytes(ctypes.byref(dims), ctypes.byref(n)))
    return n.value


def lory_moe_step_host_enqueue(dims, slot, x_host, dy_host, w_r, w1, w2, w3, y_host, dx_host, route_w_host, dw_r,
                               dw1, dw2, dw3, arena, stream=None):
    _check(load().lory_moe_step_host_enqueue(ctypes.byref(dims), int(slot), _ptr(x_host), _ptr(dy_host), _ptr(w_r),
                                             _ptr(w1), _ptr(w2), _ptr(w3), _ptr(y_host), _ptr(dx_host),
                                             _ptr(route_w_host), _ptr(dw_r), _ptr(dw1), _ptr(dw2), _ptr(dw3),
                                             _ptr(arena), _nbytes(arena), _stream(stream)))


def lory_moe_step_host_wait(slot):
    _check(load().lory_moe_step_host_wait(int(slot)))


def lory_check_status(dims, workspace, stream=None):
    _check(load().lory_check_status(ctypes.byref(dims), _ptr(workspace), _nbytes(workspace), _stream(stream)))


def lory_profile_enable(on):
    _check(load().lory_profile_enable(1 if on else 0))


def lory_profile_read(max_records=8192):
    """Returns a list of (label, milliseconds) in launch order."""
    labels = (ctypes.c_char_p * max_records)()
    ms = (ctypes.c_float * max_records)()
    n = load().lory_profile_read(max_records, labels, ms)
    if n < 0:
        _check(n)
    return [(labels[i].decode(), float(ms[i])) for i in range(n)]


LORY_NOALLOC_SCRATCH_BYTES = 4 << 20


def lory_route_noalloc(dims, x, w_r, route_w, route_p, stream=None):
    """Routing weights from x and w_r using the library's built-in scratch array (no workspace, no allocation).
    For callers whose device memory is fully handed out already; see include/lory.h for the size limit and the
    rule that calls on one device must not overlap."""
    _check(load().lory_route_noalloc(ctypes.byref(dims), _ptr(x), _ptr(w_r), _ptr(route_w), _ptr(route_p),
                                     _stream(stream)))


def lory_expert_utilization(route_w, counts, stream=None):
    """counts[e] (int32, device) = number of segments with route_w[s, e] > 2/E."""
    S, E = route_w.shape
    _check(load().lory_expert_utilization(_ptr(route_w), S, E, _ptr(counts), _stream(stream)))


def lory_selftest_bounded_wait(dims, workspace, stream=None):
    """Makes a bounded device-side wait expire on purpose; lory_check_status must then report the timeout."""
    _check(load().lory_selftest_bounded_wait(ctypes.byref(dims), _ptr(workspace), _nbytes(workspace), _stream(stream)))


def lory_probe_l2_ring(buf, slot_bytes, slots, lag, iters, mode=3, shift=0, stream=None):
    """Milliseconds of the timed pass of the write-then-read-back ring (diagnostic; see include/lory.h)."""
    ms = ctypes.c_float(0.0)
    _check(load().lory_probe_l2_ring(_ptr(buf), _nbytes(buf), int(slot_bytes), int(slots), int(lag), int(iters),
                                     int(mode), int(shift), ctypes.byref(ms), _stream(stream)))
    return ms.value


def lory_debug_build():
    """1 if the loaded library is the bounds-checking debug build, else 0."""
    return load().lory_debug_build()


def lory_selftest_debug_bounds(dims, workspace, stream=None):
    """Makes the debug build's bounds checks fire on made-up values; lory_check_status then reports them."""
    _check(load().lory_selftest_debug_bounds(ctypes.byref(dims), _ptr(workspace), _nbytes(workspace), _stream(stream)))
