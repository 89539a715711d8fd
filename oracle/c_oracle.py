"""ctypes wrapper around the C oracle (oracle/kroquant_oracle.c).

TEST INFRASTRUCTURE: see the header of the C file.  Arrays are NumPy; bf16
tensors are uint16 bit patterns.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from .build import build

_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i64, i32, vp = C.c_int64, C.c_int, C.c_void_p
        L.kq_oracle_lu_to_factors.argtypes = [vp, i32, vp]
        L.kq_oracle_lu_to_factors.restype = None
        L.kq_oracle_dense_k.argtypes = [vp, vp]
        L.kq_oracle_dense_k.restype = None
        L.kq_oracle_dense_kinv.argtypes = [vp, vp]
        L.kq_oracle_dense_kinv.restype = None
        L.kq_oracle_transform_x.argtypes = [vp, i32, i64, i32, vp, vp, i32, vp]
        L.kq_oracle_scale_transform_x.argtypes = [vp, i32, i64, i32, vp, vp]
        L.kq_oracle_widen_x.argtypes = [vp, i32, i64, i32, vp]
        L.kq_oracle_encode_block.argtypes = [vp, vp, vp]
        L.kq_oracle_encode_block.restype = None
        L.kq_oracle_mx_encode.argtypes = [vp, i64, i32, vp, vp]
        L.kq_oracle_dequantize.argtypes = [vp, vp, i64, i32, vp, i32, vp, i32]
        L.kq_oracle_hadamard_transform_x.argtypes = [vp, i32, i64, i32, vp]
        L.kq_oracle_round_y_to_16bit.argtypes = [vp, i64, i32, vp]
        L.kq_oracle_round_y_to_16bit.restype = None
        L.kq_oracle_tiled_scale_size.argtypes = [i64, i32]
        L.kq_oracle_tiled_scale_size.restype = i64
        L.kq_oracle_tiled_scale_index.argtypes = [i64, i32, i32]
        L.kq_oracle_tiled_scale_index.restype = i64
        L.kq_oracle_scales_to_tiled.argtypes = [vp, i64, i32, C.c_uint8, vp]
        L.kq_oracle_scales_to_tiled.restype = None
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _check(rc: int):
    if rc != 0:
        raise ValueError("oracle: bad shape (d must be a positive multiple of 32, "
                         "n_sets must be 1 or d/32)")


def _x(X):
    X = np.ascontiguousarray(X, dtype=np.uint16)
    assert X.ndim == 2
    return X


def _g(G):
    G = np.ascontiguousarray(G, dtype=np.float32)
    assert G.ndim == 4 and G.shape[1:] == (5, 2, 2)
    return G


def lu_to_factors(abc) -> np.ndarray:
    abc = np.ascontiguousarray(abc, dtype=np.float32)
    assert abc.ndim == 3 and abc.shape[1:] == (5, 3)
    G = np.empty((abc.shape[0], 5, 2, 2), np.float32)
    lib().kq_oracle_lu_to_factors(_p(abc), abc.shape[0], _p(G))
    return G


def dense_k(G1) -> np.ndarray:
    G1 = np.ascontiguousarray(G1, dtype=np.float32).reshape(5, 2, 2)
    K = np.empty((32, 32), np.float64)
    lib().kq_oracle_dense_k(_p(G1), _p(K))
    return K


def dense_kinv(G1) -> np.ndarray:
    G1 = np.ascontiguousarray(G1, dtype=np.float32).reshape(5, 2, 2)
    K = np.empty((32, 32), np.float64)
    lib().kq_oracle_dense_kinv(_p(G1), _p(K))
    return K


X_DTYPES = {"bf16": 0, "fp16": 1}


def transform(X, G=None, x_dtype: str = "bf16", K_dense=None) -> np.ndarray:
    """float32( x K ) per block.  Either factors G [n_sets,5,2,2] or dense K_dense [n_sets,32,32]."""
    X = _x(X)
    Y = np.empty(X.shape, np.float32)
    if K_dense is not None:
        Kd = np.ascontiguousarray(K_dense, dtype=np.float32)
        assert Kd.ndim == 3 and Kd.shape[1:] == (32, 32)
        rc = lib().kq_oracle_transform_x(_p(X), X_DTYPES[x_dtype], X.shape[0], X.shape[1], None, _p(Kd),
                                         Kd.shape[0], _p(Y))
    else:
        G = _g(G)
        rc = lib().kq_oracle_transform_x(_p(X), X_DTYPES[x_dtype], X.shape[0], X.shape[1], _p(G), None,
                                         G.shape[0], _p(Y))
    _check(rc)
    return Y


def scale_transform(X, s, x_dtype: str = "bf16") -> np.ndarray:
    X = _x(X)
    s = np.ascontiguousarray(s, dtype=np.float32)
    assert s.shape == (X.shape[1],)
    Y = np.empty(X.shape, np.float32)
    _check(lib().kq_oracle_scale_transform_x(_p(X), X_DTYPES[x_dtype], X.shape[0], X.shape[1], _p(s), _p(Y)))
    return Y


def widen(X, x_dtype: str = "bf16") -> np.ndarray:
    X = _x(X)
    Y = np.empty(X.shape, np.float32)
    _check(lib().kq_oracle_widen_x(_p(X), X_DTYPES[x_dtype], X.shape[0], X.shape[1], _p(Y)))
    return Y


def encode_block(y32) -> tuple[np.ndarray, int]:
    y = np.ascontiguousarray(y32, dtype=np.float32)
    assert y.shape == (32,)
    q = np.empty(16, np.uint8)
    s = np.empty(1, np.uint8)
    lib().kq_oracle_encode_block(_p(y), _p(q), _p(s))
    return q, int(s[0])


def mx_encode(Y) -> tuple[np.ndarray, np.ndarray]:
    Y = np.ascontiguousarray(Y, dtype=np.float32)
    t, d = Y.shape
    if d <= 0 or d % 32:
        _check(-1)
    q = np.empty((t, d // 2), np.uint8)
    s = np.empty((t, d // 32), np.uint8)
    _check(lib().kq_oracle_mx_encode(_p(Y), t, d, _p(q), _p(s)))
    return q, s


def quantize(X, G=None, x_dtype: str = "bf16", K_dense=None):
    """-> (q_packed, scales, Y) with Y the float pre-rounding values."""
    Y = transform(X, G, x_dtype, K_dense)
    q, s = mx_encode(Y)
    return q, s, Y


def scale_quantize(X, svec, x_dtype: str = "bf16"):
    Y = scale_transform(X, svec, x_dtype)
    q, s = mx_encode(Y)
    return q, s, Y


def plain_quantize(X, x_dtype: str = "bf16"):
    Y = widen(X, x_dtype)
    q, s = mx_encode(Y)
    return q, s, Y


def dequantize(q, scales, G=None, out_bf16: bool = False) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    t, half = q.shape
    d = half * 2
    assert scales.shape == (t, d // 32)
    out = np.empty((t, d), np.uint16 if out_bf16 else np.float32)
    if G is None:
        gp, ns = None, 0
    else:
        G = _g(G)
        gp, ns = _p(G), G.shape[0]
    _check(lib().kq_oracle_dequantize(_p(q), _p(scales), t, d, gp, ns, _p(out), int(out_bf16)))
    return out


def tiled_scale_index(r: int, j: int, k_blocks: int) -> int:
    return int(lib().kq_oracle_tiled_scale_index(r, j, k_blocks))


def scales_to_tiled(scales, fill: int = 0) -> np.ndarray:
    """Row-major scale bytes [rows, k_blocks] -> the 128 x 4 tiled layout block-scaled GEMMs read."""
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    rows, kb = scales.shape
    out = np.empty(int(lib().kq_oracle_tiled_scale_size(rows, kb)), np.uint8)
    lib().kq_oracle_scales_to_tiled(_p(scales), rows, kb, fill, _p(out))
    return out


def round_y_to_16bit(Y, out_dtype: str = "bf16") -> np.ndarray:
    """The transformed activations in 16 bits (uint16 patterns): float y rounded to nearest even."""
    Y = np.ascontiguousarray(Y, dtype=np.float32)
    out = np.empty(Y.shape, np.uint16)
    lib().kq_oracle_round_y_to_16bit(_p(Y), Y.size, X_DTYPES[out_dtype], _p(out))
    return out


def hadamard_transform(X, x_dtype: str = "bf16") -> np.ndarray:
    """float32( x H_d / sqrt(d) ) over the full row (d a power of two)."""
    X = _x(X)
    Y = np.empty(X.shape, np.float32)
    if lib().kq_oracle_hadamard_transform_x(_p(X), X_DTYPES[x_dtype], X.shape[0], X.shape[1], _p(Y)) != 0:
        raise ValueError("oracle: d must be a power of two >= 32")
    return Y


def hadamard_quantize(X, x_dtype: str = "bf16"):
    Y = hadamard_transform(X, x_dtype)
    q, s = mx_encode(Y)
    return q, s, Y
