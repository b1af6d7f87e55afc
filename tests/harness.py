"""Shared plumbing of the GPU parity tests: pack a synthetic layer with the library, upload it,
run the oracle on the same packed integers, and apply the acceptance tolerances."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

import oracle
from paper_2608_15531_b200 import binding as fq
from paper_2608_15531_b200 import synth

COL_TOL = 1e-2      # max |Y - Yref| <= 1e-2 * max |Yref| per output column
MEAN_TOL = 2e-3     # sum |Y - Yref| / sum |Yref|


def to_dev(a: np.ndarray) -> torch.Tensor:
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        a = a.view(np.int16)
    elif a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(a).cuda()


def bf16_bits(y: torch.Tensor) -> np.ndarray:
    return y.cpu().numpy().view(np.uint16)


def bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """binary64 -> BF16 bits, one rounding (nearest-even), via exact integer arithmetic on binary32
    is not possible in general; here used only on values that are exactly representable in binary32."""
    f = a.astype(np.float32)
    assert np.array_equal(f.astype(np.float64), a)
    u = f.view(np.uint32).astype(np.uint64)
    u = u + 0x7fff + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


@dataclass
class Packed:
    layer: synth.Layer
    L: fq.Layout
    g: int
    wq: np.ndarray
    scale: np.ndarray
    zero: np.ndarray
    indptr: np.ndarray
    info: np.ndarray
    packed: np.ndarray
    d: dict
    ws: torch.Tensor

    _q: np.ndarray | None = None

    @property
    def q(self) -> np.ndarray:
        # read back through the oracle's own format reader (cached: the matrix can be large)
        if self._q is None:
            self._q = oracle.decode_wq(self.wq, self.L.K, self.L.N, self.L.BN)
        return self._q


def pack_layer(layer: synth.Layer, g: int, BN: int = 0, upload: bool = True, value_type: int = 0) -> Packed:
    """`value_type`: type of `layer.coo_v`'s 16-bit patterns (fq.FQ_VALUE_BF16 or fq.FQ_VALUE_FP16)."""
    L = fq.fq_get_layout(layer.K, layer.N, g, bn_hint=BN)
    L.value_type = value_type
    wq, scale, zero = fq.fq_pack_int4(L, layer.W, layer.mask if layer.nnz else None)
    indptr, info, packed = fq.fq_encode_tilecoo(L, layer.coo_k, layer.coo_n, layer.coo_v)
    fq.fq_validate_tilecoo(L, indptr, info, packed)
    d, ws = {}, None
    if upload:
        pk = packed if packed.shape[0] else np.zeros((8, 16), dtype=np.uint8)
        d = dict(wq=to_dev(wq), scale=to_dev(scale), zero=to_dev(zero), indptr=to_dev(indptr), info=to_dev(info),
                 packed=to_dev(pk))
        ws = torch.zeros(fq.fq_workspace_bytes(L, fq.FQ_MAX_M), dtype=torch.uint8, device="cuda")
    return Packed(layer, L, g, wq, scale, zero, indptr, info, packed, d, ws)


def run_fused(P: Packed, X_bits: np.ndarray, streaming_only: bool = False) -> np.ndarray:
    """One fused call.  `streaming_only` sets the layout's kernel_hint for the call, so that a small layer is
    served by the streaming kernels instead of the short-job kernel the library would choose for it."""
    M = X_bits.shape[0]
    X = to_dev(X_bits)
    Y = torch.full((M, P.L.N), 0x7fc0, dtype=torch.int16, device="cuda")      # NaN pattern: every element must be written
    hint = P.L.kernel_hint
    P.L.kernel_hint = 1 if streaming_only else 0
    try:
        fq.fq_fused_w4a16_outlier_gemm(P.L, X, M, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"], P.d["info"],
                                       P.d["packed"], Y, P.ws)
        fq.fq_check_status(P.ws)
    finally:
        P.L.kernel_hint = hint
    return bf16_bits(Y)


def run_unfused(P: Packed, X_bits: np.ndarray, with_spmm: bool = True) -> np.ndarray:
    M = X_bits.shape[0]
    X = to_dev(X_bits)
    Y = torch.full((M, P.L.N), 0x7fc0, dtype=torch.int16, device="cuda")
    fq.fq_unfused_gemm(P.L, X, M, P.d["wq"], P.d["scale"], P.d["zero"], Y, P.ws)
    if with_spmm:
        fq.fq_unfused_spmm(P.L, X, M, P.d["indptr"], P.d["info"], P.d["packed"], Y)
    fq.fq_check_status(P.ws)
    return bf16_bits(Y)


def oracle_result(P: Packed, X_bits: np.ndarray, cols=None, dense_only=False):
    """Eq. 1 in binary64 on the integers the library packed (read back by the oracle's format
    readers) and the outliers as generated."""
    lay = P.layer
    if dense_only:
        e = np.zeros(0, dtype=np.uint32)
        return oracle.fused_matmul(X_bits, P.q, P.scale, P.zero, P.g, e, e, np.zeros(0, dtype=np.uint16), cols=cols,
                                   want_abs=True)
    return oracle.fused_matmul(X_bits, P.q, P.scale, P.zero, P.g, lay.coo_k, lay.coo_n, lay.coo_v, cols=cols,
                               want_abs=True, value_type=P.L.value_type)


def check_tolerances(Y_bits: np.ndarray, Yref: np.ndarray, Yabs: np.ndarray, K: int):
    """The acceptance test: per-column max error and whole-matrix mean relative error.  A column
    whose reference is nearly cancelled (possible at M = 1) passes if every element is within a
    bound derived from the sum of product magnitudes: BF16 output rounding plus FP32 accumulation."""
    Y = bits_to_f64(Y_bits)
    assert np.all(np.isfinite(Y)), "non-finite output (an element was never written?)"
    err = np.abs(Y - Yref)
    col_err = err.max(axis=0)
    col_ref = np.abs(Yref).max(axis=0)
    failing = col_err > COL_TOL * col_ref
    n_fallback = int(failing.sum())
    if n_fallback:
        bound = 2.0 ** -8 * np.abs(Yref) + K * 2.0 ** -24 * Yabs
        assert np.all(err[:, failing] <= bound[:, failing]), (
            f"{n_fallback} columns exceed 1e-2 of their column maximum and the conditioning bound")
        assert n_fallback <= max(2, Y.shape[1] // 2000), f"{n_fallback} ill-conditioned columns"
    mean_rel = err.sum() / np.abs(Yref).sum()
    assert mean_rel <= MEAN_TOL, f"mean relative error {mean_rel:.3e}"
    return dict(mean_rel=float(mean_rel), worst_col=float((col_err / np.maximum(col_ref, 1e-300)).max()),
                fallback_cols=n_fallback)
