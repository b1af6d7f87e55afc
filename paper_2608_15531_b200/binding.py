"""Thin ctypes binding of ``libfq.so`` (the C ABI declared in ``include/fq.h``).

Argument marshalling only: every step of the operator runs inside the library.
Host-side calls take numpy arrays; device-side calls take torch CUDA tensors
(torch is used for device memory and streams, nothing else).  There is no
fallback: a missing or unloadable library raises at import of the first call.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfq.so")

FQ_OK = 0
FQ_ERR_INVALID_ARG = -1
FQ_ERR_UNSUPPORTED_SHAPE = -2
FQ_ERR_BUFFER_TOO_SMALL = -3
FQ_ERR_CUDA = -4
FQ_ERR_TIMEOUT = -5
FQ_ERR_FORMAT = -6
FQ_MAX_M = 128
FQ_VALUE_BF16 = 0
FQ_VALUE_FP16 = 1

EXPORTS = [
    "fq_get_layout", "fq_pack_int4_sizes", "fq_pack_int4", "fq_unpack_int4", "fq_encode_tilecoo_sizes",
    "fq_encode_tilecoo", "fq_decode_tilecoo", "fq_validate_tilecoo", "fq_workspace_bytes",
    "fq_repurpose_pad_slots",
    "fq_fused_w4a16_outlier_gemm", "fq_fused_w4a16_outlier_gemm_noalloc", "fq_unfused_gemm", "fq_unfused_spmm", "fq_fused_host_io",
    "fq_fused_host_io_async",
    "fq_check_status", "fq_last_error",
]


class Layout(ctypes.Structure):
    _fields_ = ([(n, ctypes.c_uint32) for n in
                 ("abi", "K", "N", "group", "BK", "BN", "buckets_per_tile", "wq_interleave", "coo_unit_bytes",
                  "max_tile_packets", "max_bucket_packets", "max_tail_packets", "tilecoo_encoded", "kernel_hint",
                  "slot_order", "value_type")])


class FqError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__(f"fq status {code}: {text}")
        self.code = code


_lib = None


def lib() -> ctypes.CDLL:
    """Load ``libfq.so``; raises if it has not been built (``python -m paper_2608_15531_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_15531_b200.build`")
        _lib = ctypes.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(_lib, name).restype = ctypes.c_int32
        _lib.fq_last_error.restype = ctypes.c_char_p
    return _lib


def _check(code: int) -> None:
    if code != FQ_OK:
        raise FqError(code, lib().fq_last_error().decode(errors="replace"))


def _np(a, dtype=None):
    if a is None:
        return None
    a = np.ascontiguousarray(a) if dtype is None else np.ascontiguousarray(a, dtype=dtype)
    return a


def _hp(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else ctypes.c_void_p(0)


def _dp(t):
    """Device pointer of a torch CUDA tensor (or None)."""
    if t is None:
        return ctypes.c_void_p(0)
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


# ------------------------------------------------------------------ host, offline

def fq_get_layout(K: int, N: int, group: int, bn_hint: int = 0, nb_hint: int = 0) -> Layout:
    L = Layout()
    _check(lib().fq_get_layout(ctypes.c_uint32(K), ctypes.c_uint32(N), ctypes.c_uint32(group),
                               ctypes.c_uint32(bn_hint), ctypes.c_uint32(nb_hint), ctypes.byref(L)))
    return L


def fq_pack_int4_sizes(L: Layout):
    a, b, c = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib().fq_pack_int4_sizes(ctypes.byref(L), ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)))
    return a.value, b.value, c.value


def fq_pack_int4(L: Layout, W: np.ndarray, outlier_mask: np.ndarray | None):
    """Returns (wq uint32[K*N/8], scale uint16[G, N], zero uint16[G, N])."""
    W = _np(W, np.float32)
    assert W.shape == (L.K, L.N)
    mask = _np(outlier_mask, np.uint8)
    if mask is not None:
        assert mask.shape == (L.K, L.N)
    wq_b, s_b, z_b = fq_pack_int4_sizes(L)
    wq = np.empty(wq_b // 4, dtype=np.uint32)
    G = L.K // L.group
    scale = np.empty((G, L.N), dtype=np.uint16)
    zero = np.empty((G, L.N), dtype=np.uint16)
    _check(lib().fq_pack_int4(ctypes.byref(L), _hp(W), _hp(mask), _hp(wq), _hp(scale), _hp(zero)))
    return wq, scale, zero


def fq_repurpose_pad_slots(L: Layout, W: np.ndarray, mask: np.ndarray):
    """Returns (mask with the worst-quantised weights added where the packets have padding, number added)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    mask = np.ascontiguousarray(mask, dtype=np.uint8)
    assert W.shape == (L.K, L.N) and mask.shape == W.shape
    out = np.empty_like(mask)
    added = ctypes.c_uint64(0)
    _check(lib().fq_repurpose_pad_slots(ctypes.byref(L), _hp(W), _hp(mask), _hp(out), ctypes.byref(added)))
    return out, int(added.value)


def fq_unpack_int4(L: Layout, wq: np.ndarray) -> np.ndarray:
    wq = _np(wq)
    q = np.empty((L.K, L.N), dtype=np.uint8)
    _check(lib().fq_unpack_int4(ctypes.byref(L), _hp(wq), _hp(q)))
    return q


def fq_encode_tilecoo_sizes(L: Layout, k, n, val):
    k, n, val = _np(k, np.uint32), _np(n, np.uint32), _np(val, np.uint16)
    a, b, c = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    mx = ctypes.c_uint32(0)
    _check(lib().fq_encode_tilecoo_sizes(ctypes.byref(L), _hp(k), _hp(n), _hp(val), ctypes.c_size_t(k.shape[0]),
                                         ctypes.byref(a), ctypes.byref(b), ctypes.byref(c), ctypes.byref(mx)))
    return a.value, b.value, c.value, mx.value


def fq_encode_tilecoo(L: Layout, k, n, val):
    """Returns (tile_indptr uint32, bucket_info uint32, packed uint8[n_packets, 16]); sets L.max_tile_packets."""
    k, n, val = _np(k, np.uint32), _np(n, np.uint32), _np(val, np.uint16)
    n_ip, n_bi, n_pk, _ = fq_encode_tilecoo_sizes(L, k, n, val)
    indptr = np.empty(n_ip, dtype=np.uint32)
    info = np.empty(n_bi, dtype=np.uint32)
    packed = np.zeros((max(n_pk, 1), 16), dtype=np.uint8)
    _check(lib().fq_encode_tilecoo(ctypes.byref(L), _hp(k), _hp(n), _hp(val), ctypes.c_size_t(k.shape[0]),
                                   _hp(indptr), _hp(info), _hp(packed), ctypes.c_size_t(n_pk)))
    return indptr, info, packed[:n_pk]


def fq_decode_tilecoo(L: Layout, indptr, info, packed):
    indptr, info, packed = _np(indptr, np.uint32), _np(info, np.uint32), _np(packed, np.uint8)
    cap = max(packed.size // 4, 1)
    k = np.empty(cap, dtype=np.uint32)
    n = np.empty(cap, dtype=np.uint32)
    v = np.empty(cap, dtype=np.uint16)
    cnt = ctypes.c_size_t(cap)
    _check(lib().fq_decode_tilecoo(ctypes.byref(L), _hp(indptr), _hp(info), _hp(packed), _hp(k), _hp(n), _hp(v),
                                   ctypes.byref(cnt)))
    c = cnt.value
    return k[:c].copy(), n[:c].copy(), v[:c].copy()


def fq_validate_tilecoo(L: Layout, indptr, info, packed) -> None:
    indptr, info, packed = _np(indptr, np.uint32), _np(info, np.uint32), _np(packed, np.uint8)
    _check(lib().fq_validate_tilecoo(ctypes.byref(L), _hp(indptr), _hp(info), _hp(packed),
                                     ctypes.c_size_t(packed.size // 16)))


# ------------------------------------------------------------------------- device

def fq_workspace_bytes(L: Layout, M: int) -> int:
    b = ctypes.c_size_t(0)
    _check(lib().fq_workspace_bytes(ctypes.byref(L), ctypes.c_uint32(M), ctypes.byref(b)))
    return b.value


def fq_fused_w4a16_outlier_gemm(L: Layout, X, M: int, wq, scale, zero, tile_indptr, bucket_info, packed, Y,
                                workspace, stream=None) -> None:
    _check(lib().fq_fused_w4a16_outlier_gemm(ctypes.byref(L), _dp(X), ctypes.c_uint32(M), _dp(wq), _dp(scale),
                                             _dp(zero), _dp(tile_indptr), _dp(bucket_info), _dp(packed), _dp(Y),
                                             _dp(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                             _stream(stream)))


def fq_fused_w4a16_outlier_gemm_noalloc(L: Layout, X, M: int, wq, scale, zero, tile_indptr, bucket_info, packed, Y,
                                        stream=None) -> None:
    """The fused operator without a caller-provided workspace: for callers that may not allocate
    device memory.  Uses the scratch array built into the library (one per GPU, shared by all
    calls: do not overlap calls on different streams).  Refuses calls whose ``fq_workspace_bytes`` exceeds
    the array (FQ_ERR_BUFFER_TOO_SMALL): every call of more than 16 rows on a layer with 256-column tiles."""
    _check(lib().fq_fused_w4a16_outlier_gemm_noalloc(ctypes.byref(L), _dp(X), ctypes.c_uint32(M), _dp(wq), _dp(scale),
                                                     _dp(zero), _dp(tile_indptr), _dp(bucket_info), _dp(packed),
                                                     _dp(Y), _stream(stream)))


def fq_unfused_gemm(L: Layout, X, M: int, wq, scale, zero, Y, workspace, stream=None) -> None:
    _check(lib().fq_unfused_gemm(ctypes.byref(L), _dp(X), ctypes.c_uint32(M), _dp(wq), _dp(scale), _dp(zero), _dp(Y),
                                 _dp(workspace), ctypes.c_size_t(workspace.numel() * workspace.element_size()),
                                 _stream(stream)))


def fq_unfused_spmm(L: Layout, X, M: int, tile_indptr, bucket_info, packed, Y, stream=None) -> None:
    _check(lib().fq_unfused_spmm(ctypes.byref(L), _dp(X), ctypes.c_uint32(M), _dp(tile_indptr), _dp(bucket_info),
                                 _dp(packed), _dp(Y), _stream(stream)))


def fq_fused_host_io(L: Layout, X_host, M: int, x_dev, wq, scale, zero, tile_indptr, bucket_info, packed, y_dev,
                     Y_host, workspace, stream=None) -> None:
    """X_host / Y_host: host tensors (pinned for speed) or numpy arrays; the call returns after Y_host is filled."""
    xh = ctypes.c_void_p(X_host.data_ptr() if hasattr(X_host, "data_ptr") else X_host.ctypes.data)
    yh = ctypes.c_void_p(Y_host.data_ptr() if hasattr(Y_host, "data_ptr") else Y_host.ctypes.data)
    _check(lib().fq_fused_host_io(ctypes.byref(L), xh, ctypes.c_uint32(M), _dp(x_dev), _dp(wq), _dp(scale), _dp(zero),
                                  _dp(tile_indptr), _dp(bucket_info), _dp(packed), _dp(y_dev), yh, _dp(workspace),
                                  ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)))


def fq_fused_host_io_async(L: Layout, X_host, M: int, x_dev, wq, scale, zero, tile_indptr, bucket_info, packed, y_dev,
                           Y_host, workspace, stream=None) -> None:
    """As fq_fused_host_io, without the final wait: the caller synchronises the stream before reading Y_host
    (pinned host tensors)."""
    xh = ctypes.c_void_p(X_host.data_ptr() if hasattr(X_host, "data_ptr") else X_host.ctypes.data)
    yh = ctypes.c_void_p(Y_host.data_ptr() if hasattr(Y_host, "data_ptr") else Y_host.ctypes.data)
    _check(lib().fq_fused_host_io_async(ctypes.byref(L), xh, ctypes.c_uint32(M), _dp(x_dev), _dp(wq), _dp(scale),
                                        _dp(zero), _dp(tile_indptr), _dp(bucket_info), _dp(packed), _dp(y_dev), yh,
                                        _dp(workspace),
                                        ctypes.c_size_t(workspace.numel() * workspace.element_size()), _stream(stream)))


def fq_check_status(workspace, stream=None) -> None:
    _check(lib().fq_check_status(_dp(workspace), _stream(stream)))


def fq_last_error() -> str:
    return lib().fq_last_error().decode(errors="replace")
