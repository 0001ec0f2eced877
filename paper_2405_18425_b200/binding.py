"""Thin ctypes binding of libvig_bigla.so: argument marshalling only.

Every function mirrors the C entry point of the same name (include/vig_bigla.h), takes torch
tensors for device buffers (numpy arrays or torch CPU tensors for the host entry point), passes
their addresses and the current CUDA stream, and raises VigError on a non-zero status.  There is
no fallback: if the shared library has not been built the import of the symbols fails loudly.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libvig_bigla.so")

VIG_OK = 0
VIG_DTYPE_F32 = 0
VIG_DTYPE_BF16 = 1

_lib = None


class VigError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where} failed: status {status} ({status_string(status)})")


def load() -> ctypes.CDLL:
    """Loads the CUDA library (built in-tree by paper_2405_18425_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2405_18425_b200.build` "
                "(there is no CPU or PyTorch fallback for the BiGLA path)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
        fwd = [vp] * 6 + [ci] * 5 + [vp]
        for name in ("vig_bigla_fwd", "vig_bigla_fwd_bf16", "vig_bigla_fwd_f32", "vig_bigla_fwd_static_bf16"):
            getattr(lib, name).argtypes = fwd
            getattr(lib, name).restype = ci
        lib.vig_bigla_fwd_ws_bf16.argtypes = [vp] * 6 + [ci] * 5 + [vp, ctypes.c_size_t, vp]
        lib.vig_bigla_fwd_ws_bf16.restype = ci
        lib.vig_bigla_workspace_bytes.argtypes = [ci] * 6
        lib.vig_bigla_workspace_bytes.restype = ctypes.c_size_t
        for name in ("vig_gate_prep_bf16", "vig_gate_prep_f32"):
            getattr(lib, name).argtypes = [vp] * 4 + [ci] * 4 + [cf, vp]
            getattr(lib, name).restype = ci
        lib.vig_bigla_fwd_gates_bf16.argtypes = [vp] * 6 + [ci] * 5 + [cf, vp]
        lib.vig_bigla_fwd_gates_bf16.restype = ci
        lib.vig_bigla_fwd_blend_bf16.argtypes = [vp] * 8 + [ci] * 5 + [cf, vp]
        lib.vig_bigla_fwd_blend_bf16.restype = ci
        for name in ("vig_dwconv3x3_bf16", "vig_dwconv3x3_f32"):
            getattr(lib, name).argtypes = [vp] * 4 + [ci] * 4 + [vp]
            getattr(lib, name).restype = ci
        for name in ("vig_gate_blend_bf16", "vig_gate_blend_f32"):
            getattr(lib, name).argtypes = [vp] * 4 + [ctypes.c_longlong, vp]
            getattr(lib, name).restype = ci
        for name in ("vig_bigla_bwd_bf16", "vig_bigla_bwd_f32"):
            getattr(lib, name).argtypes = [vp] * 11 + [ci] * 5 + [vp]
            getattr(lib, name).restype = ci
        for name in ("vig_gate_prep_bwd_bf16", "vig_gate_prep_bwd_f32"):
            getattr(lib, name).argtypes = [vp] * 6 + [ci] * 4 + [cf, vp]
            getattr(lib, name).restype = ci
        lib.vig_bigla_fwd_host.argtypes = [vp] * 6 + [ci] * 5 + [cf, ci, vp]
        lib.vig_bigla_fwd_host.restype = ci
        lib.vig_status_string.argtypes = [ci]
        lib.vig_status_string.restype = ctypes.c_char_p
        lib.vig_last_device_status.argtypes = [vp]
        lib.vig_last_device_status.restype = ci
        lib.vig_test_set_kernel_preference.argtypes = [ci]
        lib.vig_test_set_kernel_preference.restype = ci
        lib.vig_test_take_fallback_count.argtypes = [vp]
        lib.vig_test_take_fallback_count.restype = ci
        lib.vig_test_expire_next_wait.argtypes = []
        lib.vig_test_expire_next_wait.restype = None
        lib.vig_kernel_launch_count.argtypes = []
        lib.vig_kernel_launch_count.restype = ctypes.c_ulonglong
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().vig_status_string(int(status)).decode()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _dims(q: torch.Tensor, v: torch.Tensor):
    B, H, L, dk = q.shape
    return B, H, L, dk, v.shape[3]


def _check(status: int, where: str):
    if status != VIG_OK:
        raise VigError(status, where)


def _dev(*tensors):
    for t in tensors:
        if not (t.is_cuda and t.is_contiguous()):
            raise ValueError("device entry points take contiguous CUDA tensors")


def vig_bigla_fwd_bf16(q, k, v, log_alpha_fwd, log_alpha_bwd, out, stream=None):
    _dev(q, k, v, log_alpha_fwd, log_alpha_bwd, out)
    _check(load().vig_bigla_fwd_bf16(q.data_ptr(), k.data_ptr(), v.data_ptr(), log_alpha_fwd.data_ptr(),
                                     log_alpha_bwd.data_ptr(), out.data_ptr(), *_dims(q, v), _stream(stream)),
           "vig_bigla_fwd_bf16")
    return out


def vig_bigla_fwd(q, k, v, log_alpha_fwd, log_alpha_bwd, out, stream=None):
    _dev(q, k, v, log_alpha_fwd, log_alpha_bwd, out)
    _check(load().vig_bigla_fwd(q.data_ptr(), k.data_ptr(), v.data_ptr(), log_alpha_fwd.data_ptr(),
                                log_alpha_bwd.data_ptr(), out.data_ptr(), *_dims(q, v), _stream(stream)),
           "vig_bigla_fwd")
    return out


def vig_bigla_fwd_f32(q, k, v, log_alpha_fwd, log_alpha_bwd, out, stream=None):
    _dev(q, k, v, log_alpha_fwd, log_alpha_bwd, out)
    _check(load().vig_bigla_fwd_f32(q.data_ptr(), k.data_ptr(), v.data_ptr(), log_alpha_fwd.data_ptr(),
                                    log_alpha_bwd.data_ptr(), out.data_ptr(), *_dims(q, v), _stream(stream)),
           "vig_bigla_fwd_f32")
    return out


def vig_bigla_fwd_static_bf16(q, k, v, log_alpha_fwd, log_alpha_bwd, out, stream=None):
    """The forward pass with the library's fixed built-in scratch: allocates nothing (see the header)."""
    _dev(q, k, v, log_alpha_fwd, log_alpha_bwd, out)
    _check(load().vig_bigla_fwd_static_bf16(q.data_ptr(), k.data_ptr(), v.data_ptr(), log_alpha_fwd.data_ptr(),
                                            log_alpha_bwd.data_ptr(), out.data_ptr(), *_dims(q, v),
                                            _stream(stream)), "vig_bigla_fwd_static_bf16")
    return out


def vig_bigla_workspace_bytes(B, H, L, dk, dv, dtype=VIG_DTYPE_BF16) -> int:
    return int(load().vig_bigla_workspace_bytes(B, H, L, dk, dv, dtype))


def vig_bigla_fwd_ws_bf16(q, k, v, log_alpha_fwd, log_alpha_bwd, out, ws, stream=None):
    _dev(q, k, v, log_alpha_fwd, log_alpha_bwd, out)
    ws_ptr = ws.data_ptr() if ws is not None else None
    ws_bytes = ws.numel() * ws.element_size() if ws is not None else 0
    _check(load().vig_bigla_fwd_ws_bf16(q.data_ptr(), k.data_ptr(), v.data_ptr(), log_alpha_fwd.data_ptr(),
                                        log_alpha_bwd.data_ptr(), out.data_ptr(), *_dims(q, v), ws_ptr, ws_bytes,
                                        _stream(stream)), "vig_bigla_fwd_ws_bf16")
    return out


def _gate_prep(fn_name, g_fwd, g_bwd, log_alpha_fwd, log_alpha_bwd, tau, stream):
    _dev(g_fwd, g_bwd, log_alpha_fwd, log_alpha_bwd)
    B, H, L, dk = g_fwd.shape
    _check(getattr(load(), fn_name)(g_fwd.data_ptr(), g_bwd.data_ptr(), log_alpha_fwd.data_ptr(),
                                    log_alpha_bwd.data_ptr(), B, H, L, dk, float(tau), _stream(stream)), fn_name)
    return log_alpha_fwd, log_alpha_bwd


def vig_gate_prep_bf16(g_fwd, g_bwd, log_alpha_fwd, log_alpha_bwd, tau=16.0, stream=None):
    return _gate_prep("vig_gate_prep_bf16", g_fwd, g_bwd, log_alpha_fwd, log_alpha_bwd, tau, stream)


def vig_gate_prep_f32(g_fwd, g_bwd, log_alpha_fwd, log_alpha_bwd, tau=16.0, stream=None):
    return _gate_prep("vig_gate_prep_f32", g_fwd, g_bwd, log_alpha_fwd, log_alpha_bwd, tau, stream)


def vig_bigla_fwd_gates_bf16(q, k, v, g_fwd, g_bwd, out, tau=16.0, stream=None):
    """Forward pass from the gate logits: log alpha = logsigmoid(g) / tau is prepared inside the call."""
    _dev(q, k, v, g_fwd, g_bwd, out)
    _check(load().vig_bigla_fwd_gates_bf16(q.data_ptr(), k.data_ptr(), v.data_ptr(), g_fwd.data_ptr(), g_bwd.data_ptr(),
                                           out.data_ptr(), *_dims(q, v), float(tau), _stream(stream)),
           "vig_bigla_fwd_gates_bf16")
    return out


def vig_bigla_fwd_blend_bf16(q, k, v, g_fwd, g_bwd, o_local, gate2d_logits, out, tau=16.0, stream=None):
    """Forward pass from the gate logits with the 2-D gate blend of Eq. 7 in the same call."""
    _dev(q, k, v, g_fwd, g_bwd, o_local, gate2d_logits, out)
    _check(load().vig_bigla_fwd_blend_bf16(q.data_ptr(), k.data_ptr(), v.data_ptr(), g_fwd.data_ptr(), g_bwd.data_ptr(),
                                           o_local.data_ptr(), gate2d_logits.data_ptr(), out.data_ptr(), *_dims(q, v),
                                           float(tau), _stream(stream)), "vig_bigla_fwd_blend_bf16")
    return out


def _by_dtype(t, stem):
    if t.dtype == torch.bfloat16:
        return stem + "_bf16"
    if t.dtype == torch.float32:
        return stem + "_f32"
    raise ValueError("bf16 or fp32 tensors only")


def vig_bigla_bwd(q, k, v, log_alpha_fwd, log_alpha_bwd, d_out, dq, dk, dv, dlog_alpha_fwd, dlog_alpha_bwd, stream=None):
    """Gradient of the forward pass (Eq. 6) for d_out = dLoss/d_out; writes and returns the five gradient tensors."""
    ts = (q, k, v, log_alpha_fwd, log_alpha_bwd, d_out, dq, dk, dv, dlog_alpha_fwd, dlog_alpha_bwd)
    _dev(*ts)
    name = _by_dtype(q, "vig_bigla_bwd")
    if any(t.dtype != q.dtype for t in ts):
        raise ValueError("all tensors of one call share a dtype")
    _check(getattr(load(), name)(*(t.data_ptr() for t in ts), *_dims(q, v), _stream(stream)), name)
    return dq, dk, dv, dlog_alpha_fwd, dlog_alpha_bwd


def vig_gate_prep_bwd(g_fwd, g_bwd, dlog_alpha_fwd, dlog_alpha_bwd, dg_fwd, dg_bwd, tau=16.0, stream=None):
    """Gradient through the gate preparation: dg = dlog_alpha * sigmoid(-g) / tau, both directions."""
    ts = (g_fwd, g_bwd, dlog_alpha_fwd, dlog_alpha_bwd, dg_fwd, dg_bwd)
    _dev(*ts)
    name = _by_dtype(g_fwd, "vig_gate_prep_bwd")
    B, H, L, dk = g_fwd.shape
    _check(getattr(load(), name)(*(t.data_ptr() for t in ts), B, H, L, dk, float(tau), _stream(stream)), name)
    return dg_fwd, dg_bwd


def vig_dwconv3x3(x, w, bias, out, stream=None):
    """Depth-wise 3x3 convolution (Eq. 7 line 1); x, out: [B, Hh, Ww, C]; w: [C, 3, 3]; bias: [C] or None."""
    _dev(x, w, out)
    name = _by_dtype(x, "vig_dwconv3x3")
    B, Hh, Ww, C = x.shape
    _check(getattr(load(), name)(x.data_ptr(), w.data_ptr(), bias.data_ptr() if bias is not None else None, out.data_ptr(),
                                 B, Hh, Ww, C, _stream(stream)), name)
    return out


def vig_gate_blend(o_local, gate2d_logits, o_global, out, stream=None):
    """out = sigmoid(z) * o_local + (1 - sigmoid(z)) * o_global, element-wise (Eq. 7 lines 3-4)."""
    _dev(o_local, gate2d_logits, o_global, out)
    name = _by_dtype(out, "vig_gate_blend")
    _check(getattr(load(), name)(o_local.data_ptr(), gate2d_logits.data_ptr(), o_global.data_ptr(), out.data_ptr(),
                                 out.numel(), _stream(stream)), name)
    return out


def _host_ptr(a) -> int:
    if isinstance(a, torch.Tensor):
        if a.is_cuda or not a.is_contiguous():
            raise ValueError("the host entry point takes contiguous CPU tensors or numpy arrays")
        return a.data_ptr()
    if not a.flags["C_CONTIGUOUS"]:
        raise ValueError("the host entry point takes C-contiguous arrays")
    return a.ctypes.data


def vig_bigla_fwd_host(q, k, v, g_fwd, g_bwd, out, tau=16.0, dtype=VIG_DTYPE_BF16, stream=None):
    """Host buffers in, host buffer out ([B,H,L,d] shapes are read from q and v)."""
    B, H, L, dk = q.shape
    dv = v.shape[3]
    _check(load().vig_bigla_fwd_host(_host_ptr(q), _host_ptr(k), _host_ptr(v), _host_ptr(g_fwd), _host_ptr(g_bwd),
                                     _host_ptr(out), B, H, L, dk, dv, float(tau), int(dtype), _stream(stream)),
           "vig_bigla_fwd_host")
    return out


def vig_last_device_status(stream=None) -> int:
    return int(load().vig_last_device_status(_stream(stream)))


VIG_TEST_KERNEL_AUTO, VIG_TEST_KERNEL_SIMT, VIG_TEST_KERNEL_CHUNK_TASKS, VIG_TEST_KERNEL_SEGMENTS = 0, 2, 3, 4


def vig_test_set_kernel_preference(preference: int) -> None:
    """Test hook (csrc/test_hooks.h; not part of the public C ABI): forces a kernel family process-wide."""
    _check(load().vig_test_set_kernel_preference(int(preference)), "vig_test_set_kernel_preference")


def vig_test_take_fallback_count(stream=None) -> int:
    """Test hook: units handed to the in-kernel recurrence since the last reading (reads and clears)."""
    return int(load().vig_test_take_fallback_count(_stream(stream)))


def vig_test_expire_next_wait() -> None:
    """Test hook: the next single-block tensor-core launch lets one bounded device-side wait run out."""
    load().vig_test_expire_next_wait()


def vig_kernel_launch_count() -> int:
    return int(load().vig_kernel_launch_count())
