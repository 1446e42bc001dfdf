"""ctypes binding of libdtst.so: argument marshalling only.

Module-level functions carry the C entry points' names and take torch CUDA
tensors where the C ABI takes device pointers.  `Plan` is a convenience wrapper
that owns the workspace tensor and allocates outputs.  Every step of the layer
runs in the library's CUDA kernels; there is no CPU or PyTorch fallback, and a
missing library is a hard error.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdtst.so")

DTST_OK = 0
DTST_ERR_INVALID_ARG = -1
DTST_ERR_UNSUPPORTED = -2
DTST_ERR_ALLOC = -3
DTST_ERR_CUDA = -4
DTST_ERR_WORKSPACE = -5
DTST_ERR_DEVICE_TIMEOUT = -6
DTST_ERR_STATIC_LIMIT = -7
DTST_STATIC_SCRATCH_BYTES = 8 * 1024 * 1024
DTST_PATH_AUTO = 0
DTST_PATH_GENERIC = 1

# every symbol include/dtst.h declares
EXPORTED = [
    "dtst_plan_create", "dtst_plan_create_local", "dtst_plan_set_virtual_shards",
    "dtst_plan_set_kernel_path", "dtst_plan_kernel_path", "dtst_plan_destroy",
    "dtst_plan_num_modes", "dtst_plan_mode_indices", "dtst_plan_workspace_bytes",
    "dtst_plan_set_workspace", "dtst_forward", "dtst_spectral_mul", "dtst_inverse",
    "dtst_backward", "dtst_plan_status", "dtst_plan_launch_count", "dtst_status_string",
    "dtst_version", "dtst_plan_enable_kernel_timing", "dtst_plan_kernel_timing", "dtst_forward_static",
    "dtst_plan_last_cuda_error", "dtst_spectral_mul_modes", "dtst_backward_spectrum", "dtst_backward_mix_modes",
    "dtst_backward_input", "dtst_plan_debug_ring_fault", "dtst_plan_set_column_expansion", "dtst_plan_require_fast_path", "dtst_block_forward", "dtst_block_backward",
    "dtst_plan_set_block_epilogue", "dtst_pointwise_linear", "dtst_pointwise_linear_scratch_bytes",
    "dtst_pointwise_linear_backward", "dtst_plan_create_complex", "dtst_forward_complex", "dtst_inverse_complex",
    "dtst_backward_complex", "dtst_plan_set_contraction_order", "dtst_plan_get_contraction_order",
    "dtst_plan_tune_contraction_order", "dtst_plan_host_io_bytes", "dtst_plan_enable_host_io", "dtst_step_host",
    "dtst_host_io_wait", "dtst_plan_set_column_contraction", "dtst_plan_set_arithmetic",
]


class DtstError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libdtst.so (once).  Raises if it has not been built: no fallback exists."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2607_14394_b200.build` "
            "(the spectral layer has no CPU or PyTorch fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64p, i32p = ctypes.c_void_p, ctypes.c_int, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_int32)
    L.dtst_plan_create.argtypes = [ctypes.POINTER(vp), i32, i64p, i32p, i32, i32, i32]
    L.dtst_plan_create_local.argtypes = [ctypes.POINTER(vp), i32, i64p, i64p, i64p, i32p, i32, i32, i32]
    L.dtst_plan_create_complex.argtypes = [ctypes.POINTER(vp), i32, i64p, i64p, i64p, i32p, i32, i32, i32]
    L.dtst_forward_complex.argtypes = [vp, vp, vp, vp]
    L.dtst_inverse_complex.argtypes = [vp, vp, vp, vp]
    L.dtst_backward_complex.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.dtst_plan_set_contraction_order.argtypes = [vp, i32p, i32]
    L.dtst_plan_get_contraction_order.argtypes = [vp, i32p]
    L.dtst_plan_tune_contraction_order.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    L.dtst_plan_set_virtual_shards.argtypes = [vp, i32]
    L.dtst_plan_set_kernel_path.argtypes = [vp, i32]
    L.dtst_plan_kernel_path.argtypes = [vp, ctypes.POINTER(i32)]
    L.dtst_plan_destroy.argtypes = [vp]
    L.dtst_plan_num_modes.argtypes = [vp, i64p, i64p]
    L.dtst_plan_mode_indices.argtypes = [vp, i32, i64p]
    L.dtst_plan_workspace_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
    L.dtst_plan_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
    L.dtst_forward.argtypes = [vp, vp, vp, vp]
    L.dtst_forward_static.argtypes = [vp, vp, vp, vp]
    L.dtst_spectral_mul.argtypes = [vp, vp, vp, vp, vp]
    L.dtst_inverse.argtypes = [vp, vp, vp, vp]
    L.dtst_backward.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.dtst_block_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    L.dtst_block_backward.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.dtst_pointwise_linear.argtypes = [i32, i32, i32, ctypes.c_int64, vp, vp, vp, vp, vp]
    L.dtst_pointwise_linear_scratch_bytes.argtypes = [i32, i32, ctypes.POINTER(ctypes.c_size_t)]
    L.dtst_pointwise_linear_backward.argtypes = [i32, i32, i32, ctypes.c_int64, vp, vp, vp, vp, vp, vp, vp,
                                                 ctypes.c_size_t, vp]
    L.dtst_spectral_mul_modes.argtypes = [vp, vp, vp, vp, ctypes.c_int64, ctypes.c_int64, vp]
    L.dtst_backward_spectrum.argtypes = [vp, vp, vp, vp]
    L.dtst_backward_mix_modes.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_int64, ctypes.c_int64, vp]
    L.dtst_backward_input.argtypes = [vp, vp, vp, vp]
    L.dtst_plan_host_io_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
    L.dtst_plan_enable_host_io.argtypes = [vp, vp, ctypes.c_size_t]
    L.dtst_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.dtst_host_io_wait.argtypes = [vp]
    L.dtst_plan_set_column_expansion.argtypes = [vp, i32]
    L.dtst_plan_set_column_contraction.argtypes = [vp, i32]
    L.dtst_plan_set_arithmetic.argtypes = [vp, i32]
    L.dtst_plan_require_fast_path.argtypes = [vp, i32]
    L.dtst_plan_set_block_epilogue.argtypes = [vp, i32]
    L.dtst_plan_debug_ring_fault.argtypes = [vp, ctypes.c_int64, ctypes.c_uint32]
    L.dtst_plan_status.argtypes = [vp, vp]
    L.dtst_plan_launch_count.argtypes = [vp, i64p]
    L.dtst_plan_enable_kernel_timing.argtypes = [vp, i32]
    L.dtst_plan_kernel_timing.argtypes = [vp, i32, i64p, ctypes.POINTER(ctypes.c_double)]
    L.dtst_plan_last_cuda_error.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_char_p)]
    L.dtst_status_string.argtypes = [i32]
    L.dtst_status_string.restype = ctypes.c_char_p
    L.dtst_version.argtypes = []
    for name in EXPORTED:
        if name not in ("dtst_status_string",):
            getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().dtst_status_string(int(status)).decode()


def _check(status: int, where: str, plan=None) -> None:
    if status != DTST_OK:
        if status == DTST_ERR_CUDA and plan is not None:
            code, text = dtst_plan_last_cuda_error(plan)
            where = f"{where} [cuda error {code}: {text}]"
        raise DtstError(status, where)


def dtst_plan_last_cuda_error(plan):
    code = ctypes.c_int(0)
    text = ctypes.c_char_p()
    lib().dtst_plan_last_cuda_error(plan, ctypes.byref(code), ctypes.byref(text))
    return int(code.value), (text.value or b"").decode()


def _i64(vals: Sequence[int]):
    return (ctypes.c_int64 * len(vals))(*[int(v) for v in vals])


def _i32(vals: Sequence[int]):
    return (ctypes.c_int32 * len(vals))(*[int(v) for v in vals])


def _ptr(t: Optional[torch.Tensor], dtype: torch.dtype, name: str) -> ctypes.c_void_p:
    if t is None:
        return ctypes.c_void_p(0)
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (the C ABI takes device pointers)")
    if t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    if isinstance(stream, torch.cuda.Stream):
        return ctypes.c_void_p(stream.cuda_stream)
    return ctypes.c_void_p(int(stream))


# ------------------------------------------------------------------ C-named entry points
def dtst_plan_create(d, N, kmax, B, C_in, C_out) -> ctypes.c_void_p:
    h = ctypes.c_void_p(0)
    _check(lib().dtst_plan_create(ctypes.byref(h), int(d), _i64(N), _i32(kmax), int(B), int(C_in), int(C_out)),
           "dtst_plan_create")
    return h


def dtst_plan_create_local(d, N_global, N_local, offset, kmax, B, C_in, C_out) -> ctypes.c_void_p:
    h = ctypes.c_void_p(0)
    _check(lib().dtst_plan_create_local(ctypes.byref(h), int(d), _i64(N_global), _i64(N_local), _i64(offset),
                                        _i32(kmax), int(B), int(C_in), int(C_out)), "dtst_plan_create_local")
    return h


def dtst_plan_create_complex(d, N_global, N_local, offset, kmax, B, C_in, C_out) -> ctypes.c_void_p:
    h = ctypes.c_void_p(0)
    _check(lib().dtst_plan_create_complex(ctypes.byref(h), int(d), _i64(N_global),
                                          None if N_local is None else _i64(N_local),
                                          None if offset is None else _i64(offset), _i32(kmax), int(B), int(C_in),
                                          int(C_out)), "dtst_plan_create_complex")
    return h


def dtst_forward_complex(plan, x, Xhat, stream=None) -> None:
    _check(lib().dtst_forward_complex(plan, _ptr(x, torch.complex64, "x"), _ptr(Xhat, torch.complex64, "Xhat"),
                                      _stream_ptr(stream)), "dtst_forward_complex", plan)


def dtst_inverse_complex(plan, Yhat, y, stream=None) -> None:
    _check(lib().dtst_inverse_complex(plan, _ptr(Yhat, torch.complex64, "Yhat"), _ptr(y, torch.complex64, "y"),
                                      _stream_ptr(stream)), "dtst_inverse_complex", plan)


def dtst_backward_complex(plan, grad_y, Xhat_saved, W, grad_x, grad_W, stream=None) -> None:
    _check(lib().dtst_backward_complex(plan, _ptr(grad_y, torch.complex64, "grad_y"),
                                       _ptr(Xhat_saved, torch.complex64, "Xhat_saved"), _ptr(W, torch.complex64, "W"),
                                       _ptr(grad_x, torch.complex64, "grad_x"), _ptr(grad_W, torch.complex64, "grad_W"),
                                       _stream_ptr(stream)), "dtst_backward_complex", plan)


def dtst_plan_set_contraction_order(plan, order) -> None:
    _check(lib().dtst_plan_set_contraction_order(plan, _i32(order), len(order)), "dtst_plan_set_contraction_order")


def dtst_plan_get_contraction_order(plan, d):
    buf = (ctypes.c_int32 * max(1, d - 1))()
    _check(lib().dtst_plan_get_contraction_order(plan, buf), "dtst_plan_get_contraction_order")
    return [int(v) for v in buf][:d - 1]


def dtst_plan_tune_contraction_order(plan):
    """Returns (bytes_before, bytes_after) of the stages behind the grid-side kernel per forward-type transform."""
    a, b = ctypes.c_double(0), ctypes.c_double(0)
    _check(lib().dtst_plan_tune_contraction_order(plan, ctypes.byref(a), ctypes.byref(b)),
           "dtst_plan_tune_contraction_order")
    return float(a.value), float(b.value)


def dtst_plan_set_virtual_shards(plan, P) -> None:
    _check(lib().dtst_plan_set_virtual_shards(plan, int(P)), "dtst_plan_set_virtual_shards")


def dtst_plan_set_kernel_path(plan, path) -> None:
    _check(lib().dtst_plan_set_kernel_path(plan, int(path)), "dtst_plan_set_kernel_path")


BLOCK_EPILOGUE = {"auto": 0, "ffma": 1, "tensor": 2}


def dtst_plan_set_block_epilogue(plan, mode) -> None:
    m = BLOCK_EPILOGUE[mode] if isinstance(mode, str) else int(mode)
    _check(lib().dtst_plan_set_block_epilogue(plan, m), "dtst_plan_set_block_epilogue")


DTST_ARITH_TF32X3, DTST_ARITH_TF32 = 0, 1


def dtst_plan_set_arithmetic(plan, mode) -> None:
    if isinstance(mode, str):
        mode = {"tf32x3": DTST_ARITH_TF32X3, "tf32": DTST_ARITH_TF32}[mode]
    _check(lib().dtst_plan_set_arithmetic(plan, int(mode)), "dtst_plan_set_arithmetic")


def dtst_plan_set_column_contraction(plan, mode) -> None:
    _check(lib().dtst_plan_set_column_contraction(plan, int(mode)), "dtst_plan_set_column_contraction")


def dtst_plan_require_fast_path(plan, required=True) -> None:
    _check(lib().dtst_plan_require_fast_path(plan, 1 if required else 0), "dtst_plan_require_fast_path")


def dtst_plan_set_column_expansion(plan, ring_columns) -> None:
    _check(lib().dtst_plan_set_column_expansion(plan, int(ring_columns)), "dtst_plan_set_column_expansion")


def dtst_plan_kernel_path(plan) -> int:
    v = ctypes.c_int(0)
    _check(lib().dtst_plan_kernel_path(plan, ctypes.byref(v)), "dtst_plan_kernel_path")
    return v.value


def dtst_plan_destroy(plan) -> None:
    _check(lib().dtst_plan_destroy(plan), "dtst_plan_destroy")


def dtst_plan_num_modes(plan, d):
    M = ctypes.c_int64(0)
    K = (ctypes.c_int64 * d)()
    _check(lib().dtst_plan_num_modes(plan, ctypes.byref(M), K), "dtst_plan_num_modes")
    return M.value, tuple(int(v) for v in K)


def dtst_plan_mode_indices(plan, dim, count):
    buf = (ctypes.c_int64 * count)()
    _check(lib().dtst_plan_mode_indices(plan, int(dim), buf), "dtst_plan_mode_indices")
    return [int(v) for v in buf]


def dtst_plan_workspace_bytes(plan) -> int:
    v = ctypes.c_size_t(0)
    _check(lib().dtst_plan_workspace_bytes(plan, ctypes.byref(v)), "dtst_plan_workspace_bytes")
    return int(v.value)


def dtst_plan_set_workspace(plan, ws: torch.Tensor) -> None:
    _check(lib().dtst_plan_set_workspace(plan, _ptr(ws, torch.uint8, "workspace"), ws.numel()),
           "dtst_plan_set_workspace")


def dtst_forward(plan, x, Xhat, stream=None) -> None:
    _check(lib().dtst_forward(plan, _ptr(x, torch.float32, "x"), _ptr(Xhat, torch.complex64, "Xhat"),
                              _stream_ptr(stream)), "dtst_forward", plan)


def dtst_forward_static(plan, x, Xhat, stream=None) -> None:
    """dtst_forward for callers that may not allocate: intermediates live in the library's fixed
    device array (DTST_STATIC_SCRATCH_BYTES), shared by all calls; no workspace is needed.
    Raises DtstError(DTST_ERR_STATIC_LIMIT) when the plan's intermediates do not fit."""
    _check(lib().dtst_forward_static(plan, _ptr(x, torch.float32, "x"), _ptr(Xhat, torch.complex64, "Xhat"),
                                     _stream_ptr(stream)), "dtst_forward_static", plan)


def dtst_spectral_mul(plan, Xhat, W, Yhat, stream=None) -> None:
    _check(lib().dtst_spectral_mul(plan, _ptr(Xhat, torch.complex64, "Xhat"), _ptr(W, torch.complex64, "W"),
                                   _ptr(Yhat, torch.complex64, "Yhat"), _stream_ptr(stream)), "dtst_spectral_mul", plan)


def dtst_inverse(plan, Yhat, y, stream=None) -> None:
    _check(lib().dtst_inverse(plan, _ptr(Yhat, torch.complex64, "Yhat"), _ptr(y, torch.float32, "y"),
                              _stream_ptr(stream)), "dtst_inverse", plan)


def dtst_backward(plan, grad_y, Xhat_saved, W, grad_x, grad_W, stream=None) -> None:
    _check(lib().dtst_backward(plan, _ptr(grad_y, torch.float32, "grad_y"),
                               _ptr(Xhat_saved, torch.complex64, "Xhat_saved"), _ptr(W, torch.complex64, "W"),
                               _ptr(grad_x, torch.float32, "grad_x"), _ptr(grad_W, torch.complex64, "grad_W"),
                               _stream_ptr(stream)), "dtst_backward", plan)


def dtst_block_forward(plan, x, W, W_bypass, out, Xhat_saved, z_saved, stream=None) -> None:
    _check(lib().dtst_block_forward(plan, _ptr(x, torch.float32, "x"), _ptr(W, torch.complex64, "W"),
                                    _ptr(W_bypass, torch.float32, "W_bypass"), _ptr(out, torch.float32, "out"),
                                    _ptr(Xhat_saved, torch.complex64, "Xhat_saved"),
                                    _ptr(z_saved, torch.float32, "z_saved"), _stream_ptr(stream)),
           "dtst_block_forward", plan)


def dtst_block_backward(plan, grad_out, x, z_saved, Xhat_saved, W, W_bypass, scratch, grad_x, grad_W, grad_W_bypass,
                        stream=None) -> None:
    _check(lib().dtst_block_backward(plan, _ptr(grad_out, torch.float32, "grad_out"), _ptr(x, torch.float32, "x"),
                                     _ptr(z_saved, torch.float32, "z_saved"),
                                     _ptr(Xhat_saved, torch.complex64, "Xhat_saved"), _ptr(W, torch.complex64, "W"),
                                     _ptr(W_bypass, torch.float32, "W_bypass"), _ptr(scratch, torch.float32, "scratch"),
                                     _ptr(grad_x, torch.float32, "grad_x"), _ptr(grad_W, torch.complex64, "grad_W"),
                                     _ptr(grad_W_bypass, torch.float32, "grad_W_bypass"), _stream_ptr(stream)),
           "dtst_block_backward", plan)


def dtst_pointwise_linear(x, W, bias, out, stream=None) -> None:
    """out[b, o, ...] = sum_i W[o, i] x[b, i, ...] + bias[o]; x [B, C_in, ...], out [B, C_out, ...]."""
    B, Ci = x.shape[0], x.shape[1]
    Co = W.shape[0]
    P = x[0, 0].numel()
    if W.shape != (Co, Ci) or out.shape[0] != B or out.shape[1] != Co or out[0, 0].numel() != P or \
            (bias is not None and bias.numel() != Co):
        raise ValueError("pointwise linear: shapes do not fit")
    with torch.cuda.device(x.device):
        _check(lib().dtst_pointwise_linear(B, Ci, Co, P, _ptr(x, torch.float32, "x"), _ptr(W, torch.float32, "W"),
                                           _ptr(bias, torch.float32, "bias"), _ptr(out, torch.float32, "out"),
                                           _stream_ptr(stream)), "dtst_pointwise_linear")


def dtst_pointwise_linear_scratch_bytes(C_in, C_out) -> int:
    v = ctypes.c_size_t(0)
    _check(lib().dtst_pointwise_linear_scratch_bytes(int(C_in), int(C_out), ctypes.byref(v)),
           "dtst_pointwise_linear_scratch_bytes")
    return int(v.value)


def dtst_pointwise_linear_backward(grad_out, x, W, grad_x, grad_W, grad_bias, scratch, stream=None) -> None:
    B, Ci = x.shape[0], x.shape[1]
    Co = W.shape[0]
    P = x[0, 0].numel()
    if W.shape != (Co, Ci) or grad_out.shape[0] != B or grad_out.shape[1] != Co or grad_out[0, 0].numel() != P or \
            (grad_x is not None and grad_x.shape != x.shape) or (grad_W is not None and grad_W.shape != W.shape) or \
            (grad_bias is not None and grad_bias.numel() != Co):
        raise ValueError("pointwise linear backward: shapes do not fit")
    with torch.cuda.device(x.device):
        _check(lib().dtst_pointwise_linear_backward(
            B, Ci, Co, P, _ptr(grad_out, torch.float32, "grad_out"), _ptr(x, torch.float32, "x"),
            _ptr(W, torch.float32, "W"), _ptr(grad_x, torch.float32, "grad_x"), _ptr(grad_W, torch.float32, "grad_W"),
            _ptr(grad_bias, torch.float32, "grad_bias"), _ptr(scratch, torch.uint8, "scratch"),
            0 if scratch is None else scratch.numel(), _stream_ptr(stream)), "dtst_pointwise_linear_backward")


def dtst_spectral_mul_modes(plan, Xhat, W_shard, Yhat_chunk, m0, count, stream=None) -> None:
    _check(lib().dtst_spectral_mul_modes(plan, _ptr(Xhat, torch.complex64, "Xhat"),
                                         _ptr(W_shard, torch.complex64, "W_shard"),
                                         _ptr(Yhat_chunk, torch.complex64, "Yhat_chunk"), int(m0), int(count),
                                         _stream_ptr(stream)), "dtst_spectral_mul_modes", plan)


def dtst_backward_spectrum(plan, grad_y, GY, stream=None) -> None:
    _check(lib().dtst_backward_spectrum(plan, _ptr(grad_y, torch.float32, "grad_y"), _ptr(GY, torch.complex64, "GY"),
                                        _stream_ptr(stream)), "dtst_backward_spectrum", plan)


def dtst_backward_mix_modes(plan, GY, Xhat_saved, W_shard, GX_chunk, grad_W_shard, m0, count, stream=None) -> None:
    _check(lib().dtst_backward_mix_modes(plan, _ptr(GY, torch.complex64, "GY"),
                                         _ptr(Xhat_saved, torch.complex64, "Xhat_saved"),
                                         _ptr(W_shard, torch.complex64, "W_shard"),
                                         _ptr(GX_chunk, torch.complex64, "GX_chunk"),
                                         _ptr(grad_W_shard, torch.complex64, "grad_W_shard"), int(m0), int(count),
                                         _stream_ptr(stream)), "dtst_backward_mix_modes", plan)


def dtst_backward_input(plan, GX, grad_x, stream=None) -> None:
    _check(lib().dtst_backward_input(plan, _ptr(GX, torch.complex64, "GX"), _ptr(grad_x, torch.float32, "grad_x"),
                                     _stream_ptr(stream)), "dtst_backward_input", plan)


def dtst_plan_debug_ring_fault(plan, withhold_after_fills, poll_limit) -> None:
    _check(lib().dtst_plan_debug_ring_fault(plan, int(withhold_after_fills), int(poll_limit)),
           "dtst_plan_debug_ring_fault")


def dtst_plan_status(plan, stream=None) -> int:
    return int(lib().dtst_plan_status(plan, _stream_ptr(stream)))


def dtst_plan_launch_count(plan) -> int:
    v = ctypes.c_int64(0)
    _check(lib().dtst_plan_launch_count(plan, ctypes.byref(v)), "dtst_plan_launch_count")
    return int(v.value)


KERNEL_KINDS = {"grid_read": 0, "grid_write": 1, "mix": 2, "mix_adjoint": 3, "block_epilogue": 4,
                "gelu_backward": 5, "bypass_backward": 6}


def dtst_plan_enable_kernel_timing(plan, capacity: int) -> None:
    _check(lib().dtst_plan_enable_kernel_timing(plan, int(capacity)), "dtst_plan_enable_kernel_timing")


def dtst_plan_kernel_timing(plan, kind):
    """(launches, total_ms) recorded for one kernel kind since the last query."""
    n = ctypes.c_int64(0)
    ms = ctypes.c_double(0.0)
    k = KERNEL_KINDS[kind] if isinstance(kind, str) else int(kind)
    _check(lib().dtst_plan_kernel_timing(plan, k, ctypes.byref(n), ctypes.byref(ms)), "dtst_plan_kernel_timing")
    return int(n.value), float(ms.value)


def dtst_version() -> int:
    return int(lib().dtst_version())


# ------------------------------------------------------------------ convenience wrapper
class Plan:
    """A truncated-spectral-layer plan plus its workspace on one CUDA device.

    N: (local) grid extents, last one contiguous; kmax: retained modes per dim.
    With N_global/offset the plan describes one rank's block (Eq. 18).
    """

    def __init__(self, N, kmax, B, C_in, C_out, N_global=None, offset=None, virtual_shards: int = 1,
                 path: str = "auto", device=None, allocate_workspace: bool = True, column_expansion: int = 0, column_contraction: int = 0,
                 complex_fields: bool = False, arithmetic: str = "tf32x3"):
        self.N = tuple(int(n) for n in N)
        self.kmax = tuple(int(k) for k in kmax)
        self.d = len(self.N)
        self.B, self.C_in, self.C_out = int(B), int(C_in), int(C_out)
        self.device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        if self.device.type != "cuda":
            raise ValueError("a Plan lives on a CUDA device")
        if self.device.index is None:
            self.device = torch.device("cuda", torch.cuda.current_device())
        self._h = None
        self.complex_fields = bool(complex_fields)
        self.grid_dtype = torch.complex64 if complex_fields else torch.float32
        with torch.cuda.device(self.device):
            if complex_fields:
                self._h = dtst_plan_create_complex(self.d, self.N if N_global is None else N_global,
                                                   None if N_global is None else self.N, offset, self.kmax, B, C_in,
                                                   C_out)
            elif N_global is None:
                self._h = dtst_plan_create(self.d, self.N, self.kmax, B, C_in, C_out)
            else:
                self._h = dtst_plan_create_local(self.d, N_global, self.N, offset, self.kmax, B, C_in, C_out)
        if path not in ("auto", "generic"):
            raise ValueError("path must be 'auto' or 'generic'")
        dtst_plan_set_kernel_path(self._h, DTST_PATH_AUTO if path == "auto" else DTST_PATH_GENERIC)
        if virtual_shards != 1:
            dtst_plan_set_virtual_shards(self._h, virtual_shards)
        if column_expansion:
            dtst_plan_set_column_expansion(self._h, column_expansion)
        if column_contraction:
            dtst_plan_set_column_contraction(self._h, column_contraction)
        if arithmetic != "tf32x3":
            dtst_plan_set_arithmetic(self._h, arithmetic)
        self.M, self.K = dtst_plan_num_modes(self._h, self.d)
        self.workspace = None
        if allocate_workspace:
            nbytes = dtst_plan_workspace_bytes(self._h)
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            with torch.cuda.device(self.device):
                dtst_plan_set_workspace(self._h, self.workspace)

    # -- introspection
    @property
    def handle(self):
        return self._h

    @property
    def kernel_path(self) -> str:
        return {DTST_PATH_AUTO: "fused", 2: "row"}.get(dtst_plan_kernel_path(self._h), "generic")

    def mode_indices(self, dim: int):
        return dtst_plan_mode_indices(self._h, dim, self.K[dim])

    def workspace_bytes(self) -> int:
        return dtst_plan_workspace_bytes(self._h)

    def launch_count(self) -> int:
        return dtst_plan_launch_count(self._h)

    def status(self, stream=None) -> int:
        return dtst_plan_status(self._h, stream)

    def enable_kernel_timing(self, capacity: int) -> None:
        dtst_plan_enable_kernel_timing(self._h, capacity)

    def kernel_timing(self, kind):
        return dtst_plan_kernel_timing(self._h, kind)

    # -- argument checks: the C ABI takes raw device pointers, so a tensor of the wrong size or on another
    # device would make the kernels read or write out of bounds; refuse it here, as a Python error
    def _numel(self, kind: str, count=None) -> int:
        import math
        pts = math.prod(self.N)
        return {"x": self.B * self.C_in * pts, "y": self.B * self.C_out * pts,
                "Xhat": self.B * self.C_in * self.M, "Yhat": self.B * self.C_out * self.M,
                "W": self.C_in * self.C_out * self.M, "Wb": self.C_in * self.C_out,
                "Xchunk": self.B * self.C_in * (count or 0), "Ychunk": self.B * self.C_out * (count or 0),
                "Wshard": self.C_in * self.C_out * (count or 0)}[kind]

    def _expect(self, t, kind: str, name: str, count=None):
        if t is None:
            return
        if not isinstance(t, torch.Tensor) or not t.is_cuda:
            raise ValueError(f"{name} must be a CUDA tensor")
        if t.device != self.device:
            raise ValueError(f"{name} is on {t.device}, the plan on {self.device}")
        want = self._numel(kind, count)
        if t.numel() != want:
            raise ValueError(f"{name} has {t.numel()} elements, the plan needs {want} ({kind})")

    def _modes(self, m0, count):
        if not (0 <= int(m0) and int(count) >= 1 and int(m0) + int(count) <= self.M):
            raise ValueError(f"mode range [{m0}, {m0}+{count}) outside [0, {self.M})")

    # -- compute (outputs allocated here unless given)
    def forward(self, x, out=None, stream=None):
        if out is None:
            out = torch.empty((self.B, self.C_in) + self.K, dtype=torch.complex64, device=self.device)
        self._expect(x, "x", "x")
        self._expect(out, "Xhat", "out")
        with torch.cuda.device(self.device):
            (dtst_forward_complex if self.complex_fields else dtst_forward)(self._h, x, out, stream)
        return out

    def forward_static(self, x, out, stream=None):
        """Forward partial DFT into the caller's `out` using only the library's fixed scratch."""
        self._expect(x, "x", "x")
        self._expect(out, "Xhat", "out")
        with torch.cuda.device(self.device):
            dtst_forward_static(self._h, x, out, stream)
        return out

    def spectral_mul(self, Xhat, W, out=None, stream=None):
        if out is None:
            out = torch.empty((self.B, self.C_out) + self.K, dtype=torch.complex64, device=self.device)
        self._expect(Xhat, "Xhat", "Xhat")
        self._expect(W, "W", "W")
        self._expect(out, "Yhat", "out")
        with torch.cuda.device(self.device):
            dtst_spectral_mul(self._h, Xhat, W, out, stream)
        return out

    def inverse(self, Yhat, out=None, stream=None):
        if out is None:
            out = torch.empty((self.B, self.C_out) + self.N, dtype=self.grid_dtype, device=self.device)
        self._expect(Yhat, "Yhat", "Yhat")
        self._expect(out, "y", "out")
        with torch.cuda.device(self.device):
            (dtst_inverse_complex if self.complex_fields else dtst_inverse)(self._h, Yhat, out, stream)
        return out

    def backward(self, grad_y, Xhat_saved, W, grad_x=None, grad_W=None, need_grad_x=True, need_grad_W=True,
                 stream=None):
        if grad_x is None and need_grad_x:
            grad_x = torch.empty((self.B, self.C_in) + self.N, dtype=self.grid_dtype, device=self.device)
        if grad_W is None and need_grad_W:
            grad_W = torch.empty((self.C_in, self.C_out, self.M), dtype=torch.complex64, device=self.device)
        self._expect(grad_y, "y", "grad_y")
        self._expect(Xhat_saved, "Xhat", "Xhat_saved")
        self._expect(W, "W", "W")
        self._expect(grad_x, "x", "grad_x")
        self._expect(grad_W, "W", "grad_W")
        with torch.cuda.device(self.device):
            (dtst_backward_complex if self.complex_fields else dtst_backward)(self._h, grad_y, Xhat_saved, W, grad_x,
                                                                               grad_W, stream)
        return grad_x, grad_W

    # -- the whole block of Algorithm 1: GELU(W_bypass x + layer(x))
    def block_forward(self, x, W, W_bypass, out=None, Xhat=None, z=None, save_z=True, stream=None):
        """Returns (out, Xhat, z); z (the pre-activation, needed by block_backward) is None with save_z=False."""
        if out is None:
            out = torch.empty((self.B, self.C_out) + self.N, dtype=torch.float32, device=self.device)
        if Xhat is None:
            Xhat = torch.empty((self.B, self.C_in) + self.K, dtype=torch.complex64, device=self.device)
        if z is None and save_z:
            z = torch.empty((self.B, self.C_out) + self.N, dtype=torch.float32, device=self.device)
        for t, kind, name in ((x, "x", "x"), (W, "W", "W"), (W_bypass, "Wb", "W_bypass"), (out, "y", "out"),
                              (Xhat, "Xhat", "Xhat"), (z, "y", "z")):
            self._expect(t, kind, name)
        with torch.cuda.device(self.device):
            dtst_block_forward(self._h, x, W, W_bypass, out, Xhat, z, stream)
        return out, Xhat, z

    def block_backward(self, grad_out, x, z, Xhat, W, W_bypass, scratch=None, grad_x=None, grad_W=None,
                       grad_W_bypass=None, stream=None):
        """Returns (grad_x, grad_W, grad_W_bypass); `scratch` ([B, C_out, n...]) receives g_z."""
        dev = self.device
        if scratch is None:
            scratch = torch.empty((self.B, self.C_out) + self.N, dtype=torch.float32, device=dev)
        if grad_x is None:
            grad_x = torch.empty((self.B, self.C_in) + self.N, dtype=torch.float32, device=dev)
        if grad_W is None:
            grad_W = torch.empty((self.C_in, self.C_out, self.M), dtype=torch.complex64, device=dev)
        if grad_W_bypass is None:
            grad_W_bypass = torch.empty((self.C_out, self.C_in), dtype=torch.float32, device=dev)
        for t, kind, name in ((grad_out, "y", "grad_out"), (x, "x", "x"), (z, "y", "z"), (Xhat, "Xhat", "Xhat"),
                              (W, "W", "W"), (W_bypass, "Wb", "W_bypass"), (scratch, "y", "scratch"),
                              (grad_x, "x", "grad_x"), (grad_W, "W", "grad_W"), (grad_W_bypass, "Wb", "grad_W_bypass")):
            self._expect(t, kind, name)
        with torch.cuda.device(self.device):
            dtst_block_backward(self._h, grad_out, x, z, Xhat, W, W_bypass, scratch, grad_x, grad_W, grad_W_bypass,
                                stream)
        return grad_x, grad_W, grad_W_bypass

    # -- the steps one by one (a rank of a slab-sharded layer exchanges spectra between them)
    def spectral_mul_modes(self, Xhat, W_shard, m0, count, out=None, stream=None):
        self._modes(m0, count)
        if out is None:
            out = torch.empty((self.B, self.C_out, count), dtype=torch.complex64, device=self.device)
        self._expect(Xhat, "Xhat", "Xhat")
        self._expect(W_shard, "Wshard", "W_shard", count)
        self._expect(out, "Ychunk", "out", count)
        with torch.cuda.device(self.device):
            dtst_spectral_mul_modes(self._h, Xhat, W_shard, out, m0, count, stream)
        return out

    def backward_spectrum(self, grad_y, out=None, stream=None):
        if out is None:
            out = torch.empty((self.B, self.C_out) + self.K, dtype=torch.complex64, device=self.device)
        self._expect(grad_y, "y", "grad_y")
        self._expect(out, "Yhat", "out")
        with torch.cuda.device(self.device):
            dtst_backward_spectrum(self._h, grad_y, out, stream)
        return out

    def backward_mix_modes(self, GY, Xhat_saved, W_shard, m0, count, GX_chunk=None, grad_W_shard=None, stream=None):
        self._modes(m0, count)
        if GX_chunk is None:
            GX_chunk = torch.empty((self.B, self.C_in, count), dtype=torch.complex64, device=self.device)
        if grad_W_shard is None:
            grad_W_shard = torch.empty((self.C_in, self.C_out, count), dtype=torch.complex64, device=self.device)
        self._expect(GY, "Yhat", "GY")
        self._expect(Xhat_saved, "Xhat", "Xhat_saved")
        self._expect(W_shard, "Wshard", "W_shard", count)
        self._expect(GX_chunk, "Xchunk", "GX_chunk", count)
        self._expect(grad_W_shard, "Wshard", "grad_W_shard", count)
        with torch.cuda.device(self.device):
            dtst_backward_mix_modes(self._h, GY, Xhat_saved, W_shard, GX_chunk, grad_W_shard, m0, count, stream)
        return GX_chunk, grad_W_shard

    def backward_input(self, GX, out=None, stream=None):
        if out is None:
            out = torch.empty((self.B, self.C_in) + self.N, dtype=torch.float32, device=self.device)
        self._expect(GX, "Xhat", "GX")
        self._expect(out, "x", "out")
        with torch.cuda.device(self.device):
            dtst_backward_input(self._h, GX, out, stream)
        return out

    def layer(self, x, W, Xhat=None, Yhat=None, y=None, stream=None):
        """y = I(M(F(x), W)); returns (y, Xhat)."""
        Xhat = self.forward(x, Xhat, stream)
        Yhat = self.spectral_mul(Xhat, W, Yhat, stream)
        y = self.inverse(Yhat, y, stream)
        return y, Xhat

    def _reset_workspace(self) -> None:
        if self.workspace is not None:
            nbytes = dtst_plan_workspace_bytes(self._h)
            if nbytes > self.workspace.numel():
                self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            with torch.cuda.device(self.device):
                dtst_plan_set_workspace(self._h, self.workspace)

    def set_contraction_order(self, order) -> None:
        """Order in which the forward-type transforms contract the dimensions 0..d-2 (a permutation)."""
        dtst_plan_set_contraction_order(self._h, order)
        self._reset_workspace()

    def contraction_order(self):
        return dtst_plan_get_contraction_order(self._h, self.d)

    def tune_contraction_order(self):
        """Most compressing dimension first; returns the modelled (bytes_before, bytes_after) of the stages."""
        r = dtst_plan_tune_contraction_order(self._h)
        self._reset_workspace()
        return r

    def set_block_epilogue(self, mode) -> None:
        """'auto', 'ffma' or 'tensor': which kernel forms the bypass product of block_forward."""
        dtst_plan_set_block_epilogue(self._h, mode)

    def set_column_contraction(self, mode: int) -> None:
        """0: automatic, 1: whenever the kernel exists for the shape, -1: never (forward-type transforms)."""
        dtst_plan_set_column_contraction(self._h, mode)

    def set_arithmetic(self, mode) -> None:
        """'tf32x3' (default: compensated, 1e-5) or 'tf32' (single pass, 2e-3) in the kernels for any extent."""
        dtst_plan_set_arithmetic(self._h, mode)

    def require_fast_path(self, required: bool = True) -> None:
        """Raises DtstError(DTST_ERR_UNSUPPORTED) if any stage of this plan would run on the slow generic kernel."""
        dtst_plan_require_fast_path(self._h, required)

    def debug_ring_fault(self, withhold_after_fills: int, poll_limit: int = 1024) -> None:
        """Diagnostic: make the forward plane kernel's bounded waits run out (see dtst_plan_debug_ring_fault)."""
        dtst_plan_debug_ring_fault(self._h, withhold_after_fills, poll_limit)

    def close(self):
        if self._h is not None:
            dtst_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class HostPipeline:
    """The whole step (F, M, I, B) for callers whose activations live in pinned HOST memory.

    A thin wrapper over `dtst_step_host`: the library chains three internal streams - copy-in, compute, copy-out -
    with events so that the PCIe transfers of x and grad_y in, and of y, grad_x and grad_W out, overlap the
    kernels and each other, also across consecutive calls of `step`.  Every byte still crosses the bus inside the
    call; nothing is cached.  W stays on the device (it is the layer's parameter).
    """

    def __init__(self, plan: Plan, W: torch.Tensor):
        self.plan, self.W = plan, W
        n = ctypes.c_size_t()
        _check(lib().dtst_plan_host_io_bytes(plan.handle, ctypes.byref(n)), "dtst_plan_host_io_bytes")
        self.staging = torch.empty(max(1, n.value), dtype=torch.uint8, device=plan.device)
        with torch.cuda.device(plan.device):
            _check(lib().dtst_plan_enable_host_io(plan.handle, _ptr(self.staging, torch.uint8, "staging"), n.value),
                   "dtst_plan_enable_host_io", plan.handle)
        self._keep = []

    def step(self, hx, hg, hy, hgx, hgW):
        """Enqueue one step; all five host tensors should be pinned.  Returns immediately; call `wait()`."""
        p = self.plan
        for t, shape, name in ((hx, (p.B, p.C_in) + p.N, "hx"), (hgx, (p.B, p.C_in) + p.N, "hgx"),
                               (hg, (p.B, p.C_out) + p.N, "hg"), (hy, (p.B, p.C_out) + p.N, "hy")):
            if t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous() or tuple(t.shape) != tuple(shape):
                raise ValueError(f"{name}: expected a contiguous float32 host tensor of shape {tuple(shape)}")
        if (hgW.is_cuda or hgW.dtype != torch.complex64 or not hgW.is_contiguous()
                or hgW.numel() != p.C_in * p.C_out * p.M):
            raise ValueError("hgW: expected a contiguous complex64 host tensor of C_in*C_out*M elements")
        p._expect(self.W, "W", "W")
        self._keep.append((hx, hg, hy, hgx, hgW))
        hp = lambda t: ctypes.c_void_p(t.data_ptr())
        with torch.cuda.device(p.device):
            _check(lib().dtst_step_host(p.handle, hp(hx), hp(hg), _ptr(self.W, torch.complex64, "W"), hp(hy), hp(hgx),
                                        hp(hgW)), "dtst_step_host", p.handle)

    def wait(self):
        _check(lib().dtst_host_io_wait(self.plan.handle), "dtst_host_io_wait", self.plan.handle)
        self._keep.clear()

    def close(self):
        if self.plan._h:
            lib().dtst_plan_enable_host_io(self.plan._h, None, 0)
