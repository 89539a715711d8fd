"""Thin ctypes binding over libkroquant.so (include/kroquant.h).

Argument marshalling only: every step of the quantizer runs in the CUDA
kernels behind the C ABI.  torch is used for device memory and streams.  There
is no CPU fallback: if the library cannot be loaded, or a call returns a
non-zero status, a :class:`KroQuantError` is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkroquant.so")

KQ_OK = 0
PATHS = {"auto": 0, "tensor": 1, "alu": 2, "onchip": 3}
EXPORTS = [
    "kroquant_factors_create", "kroquant_factors_create_lu", "kroquant_factors_create_dense",
    "kroquant_factors_destroy", "kroquant_quantize_ex", "kroquant_transform_f32_ex",
    "kroquant_scale_quantize_ex", "kroquant_mxfp4_quantize_ex", "kroquant_quantize_dual",
    "kroquant_fwht_quantize", "kroquant_fwht_transform_f32",
    "kroquant_factors_get", "kroquant_factors_n_sets", "kroquant_quantize", "kroquant_quantize_host",
    "kroquant_quantize_path", "kroquant_dequantize", "kroquant_scale_quantize",
    "kroquant_mxfp4_quantize", "kroquant_transform_f32", "kroquant_debug_e2m1_codes",
    "kroquant_tuning_default", "kroquant_quantize_tuned", "kroquant_quantize_dual_tuned", "kroquant_transform_f32_tuned",
    "kroquant_scale_quantize_tuned", "kroquant_mxfp4_quantize_tuned", "kroquant_fwht_quantize_tuned", "kroquant_debug_set_timeline", "kroquant_debug_withhold_arrival", "kroquant_debug_boundary_probe", "kroquant_launch_count", "kroquant_last_device_error",
    "kroquant_status_string",
    "kroquant_calib_create", "kroquant_calib_destroy", "kroquant_calib_set_theta", "kroquant_calib_get_theta",
    "kroquant_calib_set_lambdas", "kroquant_calib_get_lambdas", "kroquant_calib_get_factors",
    "kroquant_calib_loss_grad", "kroquant_calib_run",
    "kroquant_block_grad_scratch_bytes", "kroquant_block_grad", "kroquant_block_grad_static",
    "kroquant_calib_set_gemm_variant", "kroquant_gemm_mxfp4_variant", "kroquant_gemm_bf16_variant", "kroquant_calib_get_weight_factors", "kroquant_gemm_mxfp4",
    "kroquant_linear_w4a4", "kroquant_gemm_bf16",
]


class KroQuantError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


_lib: Optional[C.CDLL] = None


def load_library() -> C.CDLL:
    """Load libkroquant.so (built in-tree by ``paper_2607_21446_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2607_21446_b200.build` "
            "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int
    L.kroquant_factors_create.argtypes = [vp, i32, C.POINTER(vp)]
    L.kroquant_factors_create_lu.argtypes = [vp, i32, C.POINTER(vp)]
    L.kroquant_factors_create_dense.argtypes = [vp, i32, C.POINTER(vp)]
    L.kroquant_quantize_ex.argtypes = [vp, i32, i64, i32, vp, vp, vp, i32, i32, vp]
    L.kroquant_transform_f32_ex.argtypes = [vp, i32, i64, i32, vp, vp, i32, vp]
    L.kroquant_quantize_dual.argtypes = [vp, i32, i64, i32, vp, vp, vp, i32, vp, vp]
    L.kroquant_fwht_quantize.argtypes = [vp, i32, i64, i32, vp, vp, vp]
    L.kroquant_fwht_transform_f32.argtypes = [vp, i32, i64, i32, vp, vp]
    L.kroquant_scale_quantize_ex.argtypes = [vp, i32, i64, i32, vp, vp, vp, i32, vp]
    L.kroquant_mxfp4_quantize_ex.argtypes = [vp, i32, i64, i32, vp, vp, i32, vp]
    L.kroquant_factors_destroy.argtypes = [vp]
    L.kroquant_factors_destroy.restype = None
    L.kroquant_factors_get.argtypes = [vp, vp]
    L.kroquant_factors_n_sets.argtypes = [vp]
    L.kroquant_quantize.argtypes = [vp, i64, i32, vp, vp, vp, vp]
    L.kroquant_quantize_path.argtypes = [vp, i64, i32, vp, vp, vp, i32, vp]
    L.kroquant_quantize_host.argtypes = [vp, i64, i32, vp, vp, vp, vp, vp, vp, vp]
    L.kroquant_dequantize.argtypes = [vp, vp, i64, i32, vp, vp, i32, vp]
    L.kroquant_scale_quantize.argtypes = [vp, i64, i32, vp, vp, vp, vp]
    L.kroquant_mxfp4_quantize.argtypes = [vp, i64, i32, vp, vp, vp]
    L.kroquant_transform_f32.argtypes = [vp, i64, i32, vp, vp, i32, vp]
    L.kroquant_debug_e2m1_codes.argtypes = [vp, i64, vp, vp]
    L.kroquant_debug_withhold_arrival.argtypes = [i32]
    L.kroquant_tuning_default.argtypes = [vp]
    L.kroquant_tuning_default.restype = None
    L.kroquant_quantize_tuned.argtypes = [vp, i32, i64, i32, vp, vp, vp, i32, i32, vp, vp]
    L.kroquant_quantize_dual_tuned.argtypes = [vp, i32, i64, i32, vp, vp, vp, i32, vp, vp, vp]
    L.kroquant_transform_f32_tuned.argtypes = [vp, i32, i64, i32, vp, vp, i32, vp, vp]
    L.kroquant_scale_quantize_tuned.argtypes = [vp, i32, i64, i32, vp, vp, vp, i32, vp, vp]
    L.kroquant_mxfp4_quantize_tuned.argtypes = [vp, i32, i64, i32, vp, vp, i32, vp, vp]
    L.kroquant_fwht_quantize_tuned.argtypes = [vp, i32, i64, i32, vp, vp, vp, vp]
    L.kroquant_debug_set_timeline.argtypes = [vp]
    L.kroquant_debug_boundary_probe.argtypes = [i32, i32, i32, i32, i32, vp, vp]
    L.kroquant_launch_count.argtypes = []
    L.kroquant_launch_count.restype = i64
    L.kroquant_last_device_error.argtypes = [vp, C.POINTER(i32)]
    L.kroquant_status_string.argtypes = [i32]
    L.kroquant_status_string.restype = C.c_char_p
    L.kroquant_calib_create.argtypes = [vp, vp, i64, i32, i32, i32, vp, C.POINTER(vp)]
    L.kroquant_calib_destroy.argtypes = [vp]
    L.kroquant_calib_destroy.restype = None
    for name in ("set_theta", "get_theta", "set_lambdas", "get_lambdas", "get_factors", "get_weight_factors"):
        getattr(L, "kroquant_calib_" + name).argtypes = [vp, vp]
    L.kroquant_calib_loss_grad.argtypes = [vp, vp, vp, vp]
    L.kroquant_calib_run.argtypes = [vp, i32, C.c_float, vp, vp]
    L.kroquant_block_grad_scratch_bytes.argtypes = [i64, i32]
    L.kroquant_block_grad_scratch_bytes.restype = i64
    L.kroquant_block_grad.argtypes = [vp, vp, i64, i32, i32, vp, i64, vp, vp]
    L.kroquant_block_grad_static.argtypes = [vp, vp, i64, i32, i32, vp, vp]
    L.kroquant_calib_set_gemm_variant.argtypes = [vp, i32]
    L.kroquant_gemm_mxfp4_variant.argtypes = [vp, vp, vp, vp, i64, i32, i32, vp, vp, i32, i32, vp]
    L.kroquant_gemm_bf16_variant.argtypes = [vp, vp, i64, i32, i32, vp, vp, i32, i32, vp]
    L.kroquant_gemm_mxfp4.argtypes = [vp, vp, vp, vp, i64, i32, i32, vp, vp, i32, vp]
    L.kroquant_gemm_bf16.argtypes = [vp, vp, i64, i32, i32, vp, vp, i32, vp]
    L.kroquant_linear_w4a4.argtypes = [vp, i32, i64, i32, vp, vp, vp, i32, vp, vp, vp, vp, i32, vp]
    _lib = L
    return L


def status_string(status: int) -> str:
    return load_library().kroquant_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != KQ_OK:
        raise KroQuantError(status, where)


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream) if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


X_DTYPES = {torch.bfloat16: 0, torch.float16: 1}
SCALE_LAYOUTS = {"rowmajor": 0, "tiled": 1}


def tiled_scale_bytes(tokens: int, d: int) -> int:
    """Size of the scale buffer in the 128 x 4 tiled layout."""
    return ((tokens + 127) // 128) * 128 * (((d // 32) + 3) // 4) * 4


def _scale_buffer(tokens: int, d: int, layout: str, device) -> torch.Tensor:
    if layout == "tiled":      # padding bytes are never written by the kernels: start from zeros
        return torch.zeros(tiled_scale_bytes(tokens, d), dtype=torch.uint8, device=device)
    return torch.empty((tokens, max(d // 32, 0)), dtype=torch.uint8, device=device)


def _x_shape(X: torch.Tensor) -> tuple[int, int]:
    if X.dim() != 2 or X.dtype not in X_DTYPES or not X.is_cuda or not X.is_contiguous():
        raise ValueError("X must be a contiguous 2-D CUDA bfloat16 or float16 tensor [tokens, d]")
    return X.shape[0], X.shape[1]


class Factors:
    """Handle of a kroquant_factors_t.  G: float32 [n_sets, 5, 2, 2] (host)."""

    def __init__(self, handle: int, n_sets: int):
        self._h = C.c_void_p(handle)
        self.n_sets = n_sets

    @classmethod
    def create(cls, G) -> "Factors":
        G = np.ascontiguousarray(G, dtype=np.float32)
        if G.ndim != 4 or G.shape[1:] != (5, 2, 2):
            raise ValueError("G must have shape [n_sets, 5, 2, 2]")
        out = C.c_void_p()
        _check(load_library().kroquant_factors_create(G.ctypes.data_as(C.c_void_p), G.shape[0],
                                                      C.byref(out)), "kroquant_factors_create")
        return cls(out.value, G.shape[0])

    @classmethod
    def create_lu(cls, abc) -> "Factors":
        abc = np.ascontiguousarray(abc, dtype=np.float32)
        if abc.ndim != 3 or abc.shape[1:] != (5, 3):
            raise ValueError("abc must have shape [n_sets, 5, 3]")
        out = C.c_void_p()
        _check(load_library().kroquant_factors_create_lu(abc.ctypes.data_as(C.c_void_p), abc.shape[0],
                                                         C.byref(out)), "kroquant_factors_create_lu")
        return cls(out.value, abc.shape[0])

    @classmethod
    def create_dense(cls, K) -> "Factors":
        """K: float32 [n_sets, 32, 32] dense blocks, y = x K per block."""
        K = np.ascontiguousarray(K, dtype=np.float32)
        if K.ndim != 3 or K.shape[1:] != (32, 32):
            raise ValueError("K must have shape [n_sets, 32, 32]")
        out = C.c_void_p()
        _check(load_library().kroquant_factors_create_dense(K.ctypes.data_as(C.c_void_p), K.shape[0],
                                                            C.byref(out)), "kroquant_factors_create_dense")
        return cls(out.value, K.shape[0])

    def get(self) -> np.ndarray:
        G = np.empty((self.n_sets, 5, 2, 2), np.float32)
        _check(load_library().kroquant_factors_get(self._h, G.ctypes.data_as(C.c_void_p)),
               "kroquant_factors_get")
        return G

    def destroy(self) -> None:
        if self._h:
            load_library().kroquant_factors_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class Tuning(C.Structure):
    """kq_tuning_t: per-call tuning of the quantizer kernels (see include/kroquant.h).  ``Tuning()`` holds the
    library's defaults; keyword arguments override single fields."""
    _fields_ = [(n, C.c_int) for n in ("config", "ctas_per_sm", "use_pdl", "trigger", "prefetch_tiles", "dynamic",
                                       "unit_tiles", "compare_staged")]

    def __init__(self, **kw):
        super().__init__()
        load_library().kroquant_tuning_default(C.byref(self))
        for k, v in kw.items():
            if k not in dict(self._fields_):
                raise TypeError(f"unknown tuning field {k}")
            setattr(self, k, int(v))


def _tuning(t: Optional["Tuning"]):
    return None if t is None else C.cast(C.pointer(t), C.c_void_p)


def kroquant_quantize(X: torch.Tensor, factors: Factors, q_packed: Optional[torch.Tensor] = None,
                      scales: Optional[torch.Tensor] = None, path: str = "auto", stream=None,
                      scale_layout: str = "rowmajor", tuning: Optional[Tuning] = None):
    """(X bf16/fp16 [tokens, d], factors) -> (q_packed uint8 [tokens, d/2], scales uint8 [tokens, d/32]
    or, with scale_layout="tiled", a flat uint8 buffer in the 128 x 4 tiled layout)."""
    tokens, d = _x_shape(X)
    if q_packed is None:
        q_packed = torch.empty((tokens, max(d // 2, 0)), dtype=torch.uint8, device=X.device)
    if scales is None:
        scales = _scale_buffer(tokens, d, scale_layout, X.device)
    _check(load_library().kroquant_quantize_tuned(_ptr(X), X_DTYPES[X.dtype], tokens, d, factors._h, _ptr(q_packed),
                                                  _ptr(scales), SCALE_LAYOUTS[scale_layout], PATHS[path], _tuning(tuning),
                                                  C.c_void_p(_stream(stream))),
           "kroquant_quantize")
    return q_packed, scales


def kroquant_quantize_dual(X: torch.Tensor, factors: Factors, q_packed=None, scales=None, AT=None, stream=None,
                           scale_layout: str = "rowmajor", tuning: Optional[Tuning] = None):
    """One pass: MXFP4(X T) and X T itself in X's dtype -> (q_packed, scales, AT)."""
    tokens, d = _x_shape(X)
    if q_packed is None:
        q_packed = torch.empty((tokens, d // 2), dtype=torch.uint8, device=X.device)
    if scales is None:
        scales = _scale_buffer(tokens, d, scale_layout, X.device)
    if AT is None:
        AT = torch.empty_like(X)
    _check(load_library().kroquant_quantize_dual_tuned(_ptr(X), X_DTYPES[X.dtype], tokens, d, factors._h, _ptr(q_packed),
                                                       _ptr(scales), SCALE_LAYOUTS[scale_layout], _ptr(AT), _tuning(tuning),
                                                       C.c_void_p(_stream(stream))), "kroquant_quantize_dual")
    return q_packed, scales, AT


def kroquant_fwht_quantize(X: torch.Tensor, q_packed=None, scales=None, stream=None, tuning: Optional[Tuning] = None):
    """Full-d Walsh-Hadamard comparison quantizer (d a power of two, 32..16384)."""
    tokens, d = _x_shape(X)
    if q_packed is None:
        q_packed = torch.empty((tokens, d // 2), dtype=torch.uint8, device=X.device)
    if scales is None:
        scales = torch.empty((tokens, d // 32), dtype=torch.uint8, device=X.device)
    _check(load_library().kroquant_fwht_quantize_tuned(_ptr(X), X_DTYPES[X.dtype], tokens, d, _ptr(q_packed), _ptr(scales),
                                                       _tuning(tuning), C.c_void_p(_stream(stream))), "kroquant_fwht_quantize")
    return q_packed, scales


def kroquant_fwht_transform_f32(X: torch.Tensor, Y=None, stream=None):
    tokens, d = _x_shape(X)
    if Y is None:
        Y = torch.empty((tokens, d), dtype=torch.float32, device=X.device)
    _check(load_library().kroquant_fwht_transform_f32(_ptr(X), X_DTYPES[X.dtype], tokens, d, _ptr(Y),
                                                      C.c_void_p(_stream(stream))), "kroquant_fwht_transform_f32")
    return Y


def kroquant_scale_quantize(X: torch.Tensor, s: torch.Tensor, q_packed=None, scales=None, stream=None,
                            scale_layout: str = "rowmajor", tuning: Optional[Tuning] = None):
    tokens, d = _x_shape(X)
    if s.dtype != torch.float32 or not s.is_cuda or s.numel() != d or not s.is_contiguous():
        raise ValueError("s must be a contiguous CUDA float32 tensor [d]")
    if q_packed is None:
        q_packed = torch.empty((tokens, d // 2), dtype=torch.uint8, device=X.device)
    if scales is None:
        scales = _scale_buffer(tokens, d, scale_layout, X.device)
    _check(load_library().kroquant_scale_quantize_tuned(_ptr(X), X_DTYPES[X.dtype], tokens, d, _ptr(s), _ptr(q_packed),
                                                        _ptr(scales), SCALE_LAYOUTS[scale_layout], _tuning(tuning),
                                                        C.c_void_p(_stream(stream))),
           "kroquant_scale_quantize")
    return q_packed, scales


def kroquant_mxfp4_quantize(X: torch.Tensor, q_packed=None, scales=None, stream=None,
                            scale_layout: str = "rowmajor", tuning: Optional[Tuning] = None):
    tokens, d = _x_shape(X)
    if q_packed is None:
        q_packed = torch.empty((tokens, d // 2), dtype=torch.uint8, device=X.device)
    if scales is None:
        scales = _scale_buffer(tokens, d, scale_layout, X.device)
    _check(load_library().kroquant_mxfp4_quantize_tuned(_ptr(X), X_DTYPES[X.dtype], tokens, d, _ptr(q_packed),
                                                        _ptr(scales), SCALE_LAYOUTS[scale_layout], _tuning(tuning),
                                                        C.c_void_p(_stream(stream))),
           "kroquant_mxfp4_quantize")
    return q_packed, scales


def kroquant_transform_f32(X: torch.Tensor, factors: Factors, Y=None, path: str = "auto", stream=None,
                           tuning: Optional[Tuning] = None):
    tokens, d = _x_shape(X)
    if Y is None:
        Y = torch.empty((tokens, d), dtype=torch.float32, device=X.device)
    _check(load_library().kroquant_transform_f32_tuned(_ptr(X), X_DTYPES[X.dtype], tokens, d, factors._h, _ptr(Y),
                                                       PATHS[path], _tuning(tuning), C.c_void_p(_stream(stream))),
           "kroquant_transform_f32")
    return Y


def kroquant_dequantize(q_packed: torch.Tensor, scales: torch.Tensor, factors: Optional[Factors] = None,
                        out_dtype=torch.float32, out=None, stream=None):
    tokens, half = q_packed.shape
    d = half * 2
    if out is None:
        out = torch.empty((tokens, d), dtype=out_dtype, device=q_packed.device)
    code = {torch.float32: 0, torch.bfloat16: 1}[out.dtype]
    _check(load_library().kroquant_dequantize(_ptr(q_packed), _ptr(scales), tokens, d,
                                              factors._h if factors is not None else None, _ptr(out), code,
                                              C.c_void_p(_stream(stream))), "kroquant_dequantize")
    return out


def kroquant_debug_e2m1_codes(v: torch.Tensor, stream=None) -> torch.Tensor:
    codes = torch.empty(v.numel(), dtype=torch.uint8, device=v.device)
    _check(load_library().kroquant_debug_e2m1_codes(_ptr(v), v.numel(), _ptr(codes),
                                                    C.c_void_p(_stream(stream))), "kroquant_debug_e2m1_codes")
    return codes


def use_library(path: str) -> None:
    """Load another build of the library (the timeline build) instead of libkroquant.so; call before anything else."""
    global LIB_PATH, _lib
    LIB_PATH, _lib = path, None


def kroquant_debug_boundary_probe(tmem_cols: int, ctas_per_sm: int, late_trigger: bool, spin_ns: int, calls: int,
                                  marks: torch.Tensor, stream=None) -> None:
    """Diagnostic build only: `calls` chained probe launches (see the header); marks: int64 [calls, 1024, 4] on the device."""
    assert marks.dtype == torch.int64 and marks.numel() >= calls * 1024 * 4 and marks.is_cuda
    _check(load_library().kroquant_debug_boundary_probe(tmem_cols, ctas_per_sm, 1 if late_trigger else 0, spin_ns, calls,
                                                        _ptr(marks), C.c_void_p(_stream(stream))), "kroquant_debug_boundary_probe")


def kroquant_debug_set_timeline(marks: Optional[torch.Tensor]) -> None:
    _check(load_library().kroquant_debug_set_timeline(_ptr(marks)), "kroquant_debug_set_timeline")


def kroquant_debug_withhold_arrival(on: bool) -> None:
    _check(load_library().kroquant_debug_withhold_arrival(int(on)), "kroquant_debug_withhold_arrival")


def kroquant_launch_count() -> int:
    return int(load_library().kroquant_launch_count())


def kroquant_last_device_error(stream=None) -> int:
    code = C.c_int(0)
    _check(load_library().kroquant_last_device_error(C.c_void_p(_stream(stream)), C.byref(code)),
           "kroquant_last_device_error")
    return int(code.value)


# ---- host-buffer convenience used for end-to-end timing -------------------------
def quantize_from_host(X_host: torch.Tensor, factors: Factors, X_dev: torch.Tensor, q_dev: torch.Tensor,
                       s_dev: torch.Tensor, q_host: torch.Tensor, s_host: torch.Tensor, stream=None):
    """Pinned host X -> device, quantize, codes + scales -> pinned host.  All async on `stream`."""
    X_dev.copy_(X_host, non_blocking=True)
    kroquant_quantize(X_dev, factors, q_dev, s_dev, stream=stream)
    q_host.copy_(q_dev, non_blocking=True)
    s_host.copy_(s_dev, non_blocking=True)
    return q_host, s_host


def kroquant_quantize_host(X_host: torch.Tensor, factors: Factors, q_host: torch.Tensor, s_host: torch.Tensor,
                           X_work: torch.Tensor, q_work: torch.Tensor, s_work: torch.Tensor, stream=None) -> None:
    """Host tensors in, host tensors out, through the caller's device work buffers: one C call that issues the
    upload, the kernel and the two downloads in order on `stream` (asynchronous when the host tensors are pinned)."""
    tokens, d = X_host.shape
    assert X_host.dtype == torch.bfloat16 and X_host.is_contiguous() and not X_host.is_cuda
    assert q_host.shape == (tokens, d // 2) and s_host.shape == (tokens, d // 32) and not q_host.is_cuda
    assert X_work.is_cuda and X_work.shape == X_host.shape and q_work.shape == q_host.shape and s_work.shape == s_host.shape
    _check(load_library().kroquant_quantize_host(
        C.c_void_p(X_host.data_ptr()), tokens, d, factors._h, C.c_void_p(q_host.data_ptr()), C.c_void_p(s_host.data_ptr()),
        C.c_void_p(X_work.data_ptr()), C.c_void_p(q_work.data_ptr()), C.c_void_p(s_work.data_ptr()), C.c_void_p(_stream(stream))),
        "kroquant_quantize_host")


def kroquant_block_grad(X: torch.Tensor, G: torch.Tensor, n_sets: int = 1, out: Optional[torch.Tensor] = None,
                        stream=None) -> torch.Tensor:
    """out[s] = sum of x_j^T g_j over rows (and over block columns for a shared set): float32
    [n_sets, 32, 32].  X: CUDA bfloat16 [rows, d]; G: CUDA float32 [rows, d].  The scratch buffer the
    kernel needs is allocated here (torch) and passed down."""
    rows, d = _x_shape(X)
    if X.dtype != torch.bfloat16 or G.dtype != torch.float32 or G.shape != X.shape or not G.is_contiguous():
        raise ValueError("X bfloat16 [rows, d] and G float32 [rows, d], both contiguous")
    L = load_library()
    if out is None:
        out = torch.empty((n_sets, 32, 32), dtype=torch.float32, device=X.device)
    nbytes = max(int(L.kroquant_block_grad_scratch_bytes(rows, d)), 16)
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=X.device)
    _check(L.kroquant_block_grad(_ptr(X), _ptr(G), rows, d, n_sets, _ptr(scratch), nbytes, _ptr(out), _stream(stream)),
           "kroquant_block_grad")
    return out


def kroquant_block_grad_static(X: torch.Tensor, G: torch.Tensor, n_sets: int, out: torch.Tensor, stream=None) -> None:
    """kroquant_block_grad without a scratch buffer: the library's built-in one is used, so nothing is
    allocated here or below (``out``, float32 [n_sets, 32, 32], must be supplied).  For callers whose
    device memory is spoken for; see the header for the size limit and the sharing rules."""
    rows, d = _x_shape(X)
    if X.dtype != torch.bfloat16 or G.dtype != torch.float32 or G.shape != X.shape or not G.is_contiguous():
        raise ValueError("X bfloat16 [rows, d] and G float32 [rows, d], both contiguous")
    if out.dtype != torch.float32 or tuple(out.shape) != (n_sets, 32, 32) or not out.is_contiguous() or not out.is_cuda:
        raise ValueError("out must be a contiguous CUDA float32 tensor [n_sets, 32, 32]")
    _check(load_library().kroquant_block_grad_static(_ptr(X), _ptr(G), rows, d, n_sets, _ptr(out), _stream(stream)),
           "kroquant_block_grad_static")


def kroquant_gemm_mxfp4(a_codes: torch.Tensor, a_scales: torch.Tensor, b_codes: torch.Tensor, b_scales: torch.Tensor,
                        add: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                        out_dtype=torch.bfloat16, stream=None) -> torch.Tensor:
    """out[M, N] = (codes, tiled scales of A [M, K]) x (codes, tiled scales of B [N, K])^T (+ add): the W4A4
    product on the block-scaled FP4 tensor-core path.  Inputs are what the quantizer calls return with
    ``scale_layout="tiled"``."""
    for t in (a_codes, a_scales, b_codes, b_scales):
        if t.dtype != torch.uint8 or not t.is_cuda or not t.is_contiguous():
            raise ValueError("codes and scales must be contiguous CUDA uint8 tensors")
    M, half = a_codes.shape
    N = b_codes.shape[0]
    if b_codes.shape[1] != half:
        raise ValueError("A and B must share K")
    K = 2 * half
    if a_scales.numel() != tiled_scale_bytes(M, K) or b_scales.numel() != tiled_scale_bytes(N, K):
        raise ValueError("scales must be in the tiled layout (tiled_scale_bytes(rows, K) bytes)")
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=a_codes.device)
    if out.dtype not in (torch.bfloat16, torch.float32) or tuple(out.shape) != (M, N) or not out.is_contiguous():
        raise ValueError("out must be a contiguous bfloat16 or float32 tensor [M, N]")
    if add is not None and (add.dtype != torch.bfloat16 or tuple(add.shape) != (M, N) or not add.is_contiguous()):
        raise ValueError("add must be a contiguous bfloat16 tensor [M, N]")
    _check(load_library().kroquant_gemm_mxfp4_variant(_ptr(a_codes), _ptr(a_scales), _ptr(b_codes), _ptr(b_scales), M, N, K,
                                                      _ptr(add), _ptr(out), 1 if out.dtype == torch.bfloat16 else 0,
                                                      int(_GEMM_PAIR), _stream(stream)), "kroquant_gemm_mxfp4")
    return out


def kroquant_gemm_bf16(A: torch.Tensor, Bm: torch.Tensor, add: Optional[torch.Tensor] = None,
                       out: Optional[torch.Tensor] = None, out_dtype=torch.bfloat16, stream=None) -> torch.Tensor:
    """out[M, N] = A[M, K] @ Bm[N, K]^T (+ add, float32): bf16 operands, fp32 accumulation, on this library's
    tensor-core GEMM (for the 16-bit low-rank branch of the quantized layer)."""
    for t in (A, Bm):
        if t.dim() != 2 or t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
            raise ValueError("A and Bm must be contiguous 2-D CUDA bfloat16 tensors")
    M, K = A.shape
    N = Bm.shape[0]
    if Bm.shape[1] != K:
        raise ValueError("A [M, K] and Bm [N, K] must share K")
    if out is None:
        out = torch.empty((M, N), dtype=out_dtype, device=A.device)
    if out.dtype not in (torch.bfloat16, torch.float32) or tuple(out.shape) != (M, N) or not out.is_contiguous():
        raise ValueError("out must be a contiguous bfloat16 or float32 tensor [M, N]")
    if add is not None and (add.dtype != torch.float32 or tuple(add.shape) != (M, N) or not add.is_contiguous()):
        raise ValueError("add must be a contiguous float32 tensor [M, N]")
    _check(load_library().kroquant_gemm_bf16_variant(_ptr(A), _ptr(Bm), M, N, K, _ptr(add), _ptr(out),
                                                     1 if out.dtype == torch.bfloat16 else 0, int(_GEMM_PAIR),
                                                     _stream(stream)), "kroquant_gemm_bf16")
    return out


class LinearW4A4:
    """The quantized linear layer of Section 3.4: holds the activation factors, the offline-quantized
    weights (codes + tiled scales) and the work buffers for Q(X T); ``__call__`` runs quantizer + FP4 GEMM
    (two launches, nothing allocated after the first call for a given number of tokens)."""

    def __init__(self, factors: "Factors", w_codes: torch.Tensor, w_scales: torch.Tensor):
        self.factors, self.w_codes, self.w_scales = factors, w_codes, w_scales
        self.o, self.d = w_codes.shape[0], 2 * w_codes.shape[1]
        self._work = {}

    @classmethod
    def from_weights(cls, W: torch.Tensor, G_act, G_weight) -> "LinearW4A4":
        """W: CUDA bf16 [o, d]; G_act / G_weight: factor sets [n_sets, 5, 2, 2] of T and T^-T."""
        fw = Factors.create(G_weight)
        q, s = kroquant_quantize(W, fw, scale_layout="tiled")
        torch.cuda.current_stream().synchronize()
        fw.destroy()
        return cls(Factors.create(G_act), q, s)

    def __call__(self, X: torch.Tensor, add: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
                 out_dtype=torch.bfloat16, stream=None) -> torch.Tensor:
        tokens, d = _x_shape(X)
        if d != self.d:
            raise ValueError("X [tokens, d] does not match the weights")
        if tokens not in self._work:
            self._work[tokens] = (torch.empty((tokens, d // 2), dtype=torch.uint8, device=X.device),
                                  torch.zeros(tiled_scale_bytes(tokens, d), dtype=torch.uint8, device=X.device))
        q, s = self._work[tokens]
        if out is None:
            out = torch.empty((tokens, self.o), dtype=out_dtype, device=X.device)
        _check(load_library().kroquant_linear_w4a4(
            _ptr(X), X_DTYPES[X.dtype], tokens, d, self.factors._h, _ptr(self.w_codes), _ptr(self.w_scales), self.o,
            _ptr(q), _ptr(s), _ptr(add), _ptr(out), 1 if out.dtype == torch.bfloat16 else 0, _stream(stream)),
            "kroquant_linear_w4a4")
        return out


_GEMM_PAIR = True


def set_gemm_pair(on: bool) -> None:
    """Which GEMM variant THIS BINDING passes with its calls from now on (a default of the Python layer, handed to
    the library per call or per calibration handle; the library keeps no process-wide switch): pairs of CTAs on
    256 x 256 tiles (default) or one CTA per tile."""
    global _GEMM_PAIR
    _GEMM_PAIR = bool(on)


class Calibrator:
    """Handle of a kroquant_calib_t: layer-wise calibration of the transform (Section 3.3).

    A [M, d] and W [o, d] are contiguous CUDA bfloat16 tensors; they are kept alive by this object.
    """

    def __init__(self, A: torch.Tensor, W: torch.Tensor, n_sets: int = 1, stream=None):
        for t in (A, W):
            if t.dim() != 2 or t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
                raise ValueError("A and W must be contiguous 2-D CUDA bfloat16 tensors")
        if A.shape[1] != W.shape[1]:
            raise ValueError("A [M, d] and W [o, d] must share d")
        self.A, self.W, self.n_sets = A, W, n_sets
        self.M, self.d, self.o = A.shape[0], A.shape[1], W.shape[0]
        out = C.c_void_p()
        _check(load_library().kroquant_calib_create(_ptr(A), _ptr(W), self.M, self.o, self.d, n_sets,
                                                    _stream(stream), C.byref(out)), "kroquant_calib_create")
        self._h = out

    def destroy(self) -> None:
        if getattr(self, "_h", None):
            load_library().kroquant_calib_destroy(self._h)
            self._h = None

    __del__ = destroy

    def _get(self, name: str, shape) -> np.ndarray:
        out = np.empty(shape, np.float32)
        _check(getattr(load_library(), "kroquant_calib_get_" + name)(self._h, out.ctypes.data_as(C.c_void_p)),
               "kroquant_calib_get_" + name)
        return out

    @property
    def theta(self) -> np.ndarray:
        return self._get("theta", (self.n_sets, 5, 3))

    @theta.setter
    def theta(self, value) -> None:
        v = np.ascontiguousarray(value, dtype=np.float32)
        if v.shape != (self.n_sets, 5, 3):
            raise ValueError("theta must have shape [n_sets, 5, 3]")
        _check(load_library().kroquant_calib_set_theta(self._h, v.ctypes.data_as(C.c_void_p)), "kroquant_calib_set_theta")

    @property
    def lambdas(self) -> np.ndarray:
        return self._get("lambdas", (2,))

    @lambdas.setter
    def lambdas(self, value) -> None:
        v = np.ascontiguousarray(value, dtype=np.float32)
        if v.shape != (2,):
            raise ValueError("lambdas = (lambda_A, lambda_W)")
        _check(load_library().kroquant_calib_set_lambdas(self._h, v.ctypes.data_as(C.c_void_p)),
               "kroquant_calib_set_lambdas")

    def factors(self) -> np.ndarray:
        """G [n_sets, 5, 2, 2] of the current parameters (input of Factors.create)."""
        return self._get("factors", (self.n_sets, 5, 2, 2))

    def weight_factors(self) -> np.ndarray:
        """H [n_sets, 5, 2, 2] with H_k = G_k^-T: the Kronecker set of T^-T, for quantizing W offline."""
        return self._get("weight_factors", (self.n_sets, 5, 2, 2))

    def loss_grad(self, grad: bool = True, stream=None):
        """-> (losses float64 [3] = (L_out, L_A, L_W), dL/dtheta float32 [n_sets, 5, 3] or None)."""
        losses = np.empty(3, np.float64)
        g = np.empty((self.n_sets, 5, 3), np.float32) if grad else None
        _check(load_library().kroquant_calib_set_gemm_variant(self._h, int(_GEMM_PAIR)), "kroquant_calib_set_gemm_variant")
        _check(load_library().kroquant_calib_loss_grad(self._h, losses.ctypes.data_as(C.c_void_p),
                                                       g.ctypes.data_as(C.c_void_p) if grad else None,
                                                       _stream(stream)), "kroquant_calib_loss_grad")
        return losses, g

    def run(self, steps: int, lr: float = 1e-2, history: bool = True, stream=None):
        """`steps` Adam steps; -> history float64 [steps + 1, 3] (or None, asynchronous)."""
        h = np.empty((steps + 1, 3), np.float64) if history else None
        _check(load_library().kroquant_calib_set_gemm_variant(self._h, int(_GEMM_PAIR)), "kroquant_calib_set_gemm_variant")
        _check(load_library().kroquant_calib_run(self._h, steps, lr, h.ctypes.data_as(C.c_void_p) if history else None,
                                                 _stream(stream)), "kroquant_calib_run")
        return h
