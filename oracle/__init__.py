"""ctypes front-end of the CPU oracle (``fq_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline / reference arm.  The CUDA library and its Python
binding never import this package, and this package never imports them.

Arrays are numpy; BF16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fq_oracle.c")
_LIB = os.path.join(_HERE, "libfq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct)) if a is not None else None


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.orc_f32_to_bf16.restype = ctypes.c_uint16
        _lib.orc_f32_to_bf16.argtypes = [ctypes.c_float]
        _lib.orc_bf16_to_f32.restype = ctypes.c_float
        _lib.orc_bf16_to_f32.argtypes = [ctypes.c_uint16]
        _lib.orc_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def f32_to_bf16(x: float) -> int:
    return int(lib().orc_f32_to_bf16(ctypes.c_float(x)))


def bf16_to_f32(h: int) -> float:
    return float(lib().orc_bf16_to_f32(ctypes.c_uint16(h)))


def quantize(W: np.ndarray, mask: np.ndarray | None, g: int):
    """Eq. 2 per (group, column).  Returns (q uint8 KxN, scale uint16 GxN, zero uint16 GxN)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    K, N = W.shape
    if mask is not None:
        mask = np.ascontiguousarray(mask, dtype=np.uint8)
        assert mask.shape == (K, N)
    q = np.empty((K, N), dtype=np.uint8)
    s = np.empty((K // g, N), dtype=np.uint16)
    z = np.empty((K // g, N), dtype=np.uint16)
    rc = lib().orc_quantize(_p(W, ctypes.c_float), _p(mask, ctypes.c_uint8), ctypes.c_uint32(K),
                            ctypes.c_uint32(N), ctypes.c_uint32(g), _p(q, ctypes.c_uint8),
                            _p(s, ctypes.c_uint16), _p(z, ctypes.c_uint16))
    if rc != 0:
        raise ValueError(f"orc_quantize failed: {rc}")
    return q, s, z


def repurpose_pads(W: np.ndarray, mask: np.ndarray, g: int, BN: int) -> np.ndarray:
    """Section 3.2.1's remark on padding slots: the mask with, per tile, bucket and column, as many of the
    column's worst-quantised weights added as the column-slotted packets have padding for."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    K, N = W.shape
    q, s, z = quantize(W, mask, g)
    out = np.empty((K, N), dtype=np.uint8)
    lib().orc_repurpose_pads.restype = ctypes.c_int64
    rc = lib().orc_repurpose_pads(_p(W, ctypes.c_float), _p(mask, ctypes.c_uint8), ctypes.c_uint32(K),
                                  ctypes.c_uint32(N), ctypes.c_uint32(g), ctypes.c_uint32(BN),
                                  _p(q, ctypes.c_uint8), _p(s, ctypes.c_uint16), _p(z, ctypes.c_uint16),
                                  _p(out, ctypes.c_uint8))
    if rc < 0:
        raise ValueError(f"orc_repurpose_pads failed: {rc}")
    return out


def dequant(q: np.ndarray, s: np.ndarray, z: np.ndarray, g: int) -> np.ndarray:
    """Eq. 3 in binary64: What = s * (q - z)."""
    q = np.ascontiguousarray(q, dtype=np.uint8)
    s = np.ascontiguousarray(s, dtype=np.uint16)
    z = np.ascontiguousarray(z, dtype=np.uint16)
    K, N = q.shape
    out = np.empty((K, N), dtype=np.float64)
    lib().orc_dequant(_p(q, ctypes.c_uint8), _p(s, ctypes.c_uint16), _p(z, ctypes.c_uint16),
                      ctypes.c_uint32(K), ctypes.c_uint32(N), ctypes.c_uint32(g),
                      _p(out, ctypes.c_double))
    return out


def fused_matmul(X: np.ndarray, q, s, z, g: int, coo_k, coo_n, coo_v, cols=None, want_abs=False, value_type: int = 0):
    """Eq. 1 in binary64.  X: uint16 (BF16 bits) MxK.  ``coo_v``: uint16 value bits, BF16 (``value_type`` 0)
    or IEEE binary16 (1).  ``cols``: optional list of
    output columns to evaluate (all when None).  Returns Y (M x ncols) and,
    when ``want_abs``, the sum of product magnitudes."""
    X = np.ascontiguousarray(X, dtype=np.uint16)
    q = np.ascontiguousarray(q, dtype=np.uint8)
    s = np.ascontiguousarray(s, dtype=np.uint16)
    z = np.ascontiguousarray(z, dtype=np.uint16)
    M, K = X.shape
    K2, N = q.shape
    assert K2 == K
    coo_k = np.ascontiguousarray(coo_k, dtype=np.uint32)
    coo_n = np.ascontiguousarray(coo_n, dtype=np.uint32)
    coo_v = np.ascontiguousarray(coo_v, dtype=np.uint16)
    nnz = coo_k.shape[0]
    if cols is not None:
        cols = np.ascontiguousarray(cols, dtype=np.uint32)
        ncols = cols.shape[0]
    else:
        ncols = N
    Y = np.empty((M, ncols), dtype=np.float64)
    Yabs = np.empty((M, ncols), dtype=np.float64) if want_abs else None
    lib().orc_fused_matmul(_p(X, ctypes.c_uint16), ctypes.c_uint32(M), ctypes.c_uint32(K),
                           ctypes.c_uint32(N), ctypes.c_uint32(g), _p(q, ctypes.c_uint8),
                           _p(s, ctypes.c_uint16), _p(z, ctypes.c_uint16),
                           _p(coo_k, ctypes.c_uint32), _p(coo_n, ctypes.c_uint32),
                           _p(coo_v, ctypes.c_uint16), ctypes.c_uint32(value_type), ctypes.c_size_t(nnz),
                           _p(cols, ctypes.c_uint32), ctypes.c_uint32(ncols),
                           _p(Y, ctypes.c_double), _p(Yabs, ctypes.c_double))
    return (Y, Yabs) if want_abs else Y


def decode_wq(wq: np.ndarray, K: int, N: int, BN: int) -> np.ndarray:
    """Packed INT4 buffer -> q[K][N] (one code per byte), from the format description."""
    wq = np.ascontiguousarray(wq).view(np.uint32)
    assert wq.size == K * N // 8
    q = np.empty((K, N), dtype=np.uint8)
    rc = lib().orc_decode_wq(_p(wq, ctypes.c_uint32), ctypes.c_uint32(K), ctypes.c_uint32(N),
                             ctypes.c_uint32(BN), _p(q, ctypes.c_uint8))
    if rc != 0:
        raise ValueError(f"orc_decode_wq failed: {rc}")
    return q


def decode_tilecoo(tile_indptr, bucket_info, packed, K: int, N: int, BN: int, NB: int, value_type: int = 0):
    """Tile-COO arrays -> (k, n, value bits, bucket id) of every real entry; the value bits as uint16 in the
    given type (0: BF16, 1: IEEE binary16).  A value the type cannot hold exactly raises."""
    tile_indptr = np.ascontiguousarray(tile_indptr, dtype=np.uint32)
    bucket_info = np.ascontiguousarray(bucket_info, dtype=np.uint32)
    packed = np.ascontiguousarray(packed).view(np.uint8)
    npk = packed.size // 16
    cap = max(4 * npk, 1)
    k = np.empty(cap, dtype=np.uint32)
    n = np.empty(cap, dtype=np.uint32)
    v = np.empty(cap, dtype=np.uint32)
    b = np.empty(cap, dtype=np.uint32)
    cnt = ctypes.c_size_t(0)
    rc = lib().orc_decode_tilecoo(_p(tile_indptr, ctypes.c_uint32), _p(bucket_info, ctypes.c_uint32),
                                  _p(packed, ctypes.c_uint8), ctypes.c_uint32(K), ctypes.c_uint32(N),
                                  ctypes.c_uint32(BN), ctypes.c_uint32(NB), _p(k, ctypes.c_uint32),
                                  _p(n, ctypes.c_uint32), _p(v, ctypes.c_uint32),
                                  _p(b, ctypes.c_uint32), ctypes.byref(cnt))
    if rc != 0:
        raise ValueError(f"orc_decode_tilecoo failed: {rc}")
    c = cnt.value
    field = v[:c].copy()                                  # 19 bits: an FP32 number cut to ten fraction bits
    if value_type == 0:
        if (field & 7).any():
            raise ValueError("a value does not fit BF16")
        bits = (field >> 3).astype(np.uint16)
    else:
        f32 = (field << 13).view(np.float32)
        with np.errstate(over="ignore"):
            h = f32.astype(np.float16)
        if not np.array_equal(h.astype(np.float32).view(np.uint32), f32.view(np.uint32)):
            raise ValueError("a value does not fit IEEE binary16")
        bits = h.view(np.uint16)
    return k[:c].copy(), n[:c].copy(), bits, b[:c].copy()
