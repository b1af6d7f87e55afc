"""Seeded synthetic layers for the W4A16 + outlier decode matmul.

Draws numbers only (``csrc/fq_synth.c``): dense weights ~ N(0, 0.02^2) in
binary32, activations ~ N(0, 1) rounded to BF16, outlier positions in one of
three layouts, outlier magnitudes 6-20 sigma with random sign kept in BF16.
None of the method's arithmetic lives here; the CUDA library's callers and the
CPU oracle's callers both consume these arrays.

Stand-in for the paper's workloads (operator shapes taken from LLM families,
INT4 weights with 1-5 % BF16 outliers): trained weights are not available, so
shapes follow the LLaMA-3 8B / 70B linear layers and values follow the recipe
above.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csrc", "fq_synth.c")
_LIB = os.path.join(_HERE, "libfq_synth.so")
_lib = None

BASE_SEED = 260815531
SIGMA = 0.02
LAYOUTS = {"uniform": 0, "mixed": 1, "clustered": 2}


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC,
                        "-lm"], check=True)
    return _LIB


def _get():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.syn_outlier_positions.restype = ctypes.c_uint64
        _lib.syn_outlier_values.restype = ctypes.c_uint64
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


@dataclass
class Layer:
    """One synthetic linear layer: W (K x N binary32, outliers written in),
    mask (K x N uint8), outliers as COO (k, n, BF16 bits), and bookkeeping."""
    K: int
    N: int
    W: np.ndarray
    mask: np.ndarray
    coo_k: np.ndarray
    coo_n: np.ndarray
    coo_v: np.ndarray
    density: float
    layout: str
    hot_fraction: float
    seed: int

    @property
    def nnz(self) -> int:
        return int(self.coo_k.shape[0])


def tensor_seed(config: int, layer: int) -> int:
    return BASE_SEED + 1000 * config + layer


def activations(seed: int, M: int, K: int) -> np.ndarray:
    """X = bf16(N(0,1)), M x K, returned as uint16 bit patterns.  Rows are a
    prefix-stable sequence: the first rows of a larger M equal a smaller M's."""
    X = np.empty((M, K), dtype=np.uint16)
    _get().syn_activations(ctypes.c_uint64(seed), ctypes.c_uint64(M * K), _p(X, ctypes.c_uint16))
    return X


def layer(seed: int, K: int, N: int, density: float = 0.01, layout: str = "mixed",
          sigma: float = SIGMA) -> Layer:
    lib = _get()
    W = np.empty((K, N), dtype=np.float32)
    lib.syn_dense_weights(ctypes.c_uint64(seed), ctypes.c_uint64(K * N), ctypes.c_double(sigma),
                          _p(W, ctypes.c_float))
    mask = np.zeros((K, N), dtype=np.uint8)
    nnz = int(round(density * K * N))
    in_hot = 0
    if nnz > 0:
        in_hot = int(lib.syn_outlier_positions(ctypes.c_uint64(seed), ctypes.c_uint32(K),
                                               ctypes.c_uint32(N), ctypes.c_uint64(nnz),
                                               ctypes.c_int(LAYOUTS[layout]), _p(mask, ctypes.c_uint8)))
    ck = np.empty(max(nnz, 1), dtype=np.uint32)
    cn = np.empty(max(nnz, 1), dtype=np.uint32)
    cv = np.empty(max(nnz, 1), dtype=np.uint16)
    cnt = 0
    if nnz > 0:
        cnt = int(lib.syn_outlier_values(ctypes.c_uint64(seed), ctypes.c_uint32(K), ctypes.c_uint32(N),
                                         ctypes.c_double(sigma), _p(mask, ctypes.c_uint8),
                                         _p(W, ctypes.c_float), _p(ck, ctypes.c_uint32),
                                         _p(cn, ctypes.c_uint32), _p(cv, ctypes.c_uint16)))
        assert cnt == nnz
    return Layer(K=K, N=N, W=W, mask=mask, coo_k=ck[:cnt].copy(), coo_n=cn[:cnt].copy(),
                 coo_v=cv[:cnt].copy(), density=density, layout=layout,
                 hot_fraction=(in_hot / nnz if nnz else 0.0), seed=seed)


def bf16_bits_to_f32(a: np.ndarray) -> np.ndarray:
    """Widen BF16 bit patterns to binary32 (exact)."""
    return (a.astype(np.uint32) << 16).view(np.float32)


# BASELINE configurations: (name, K, N)
LLAMA3_8B = [("qkv", 4096, 6144), ("o_proj", 4096, 4096), ("gate_up", 4096, 28672), ("down", 14336, 4096)]
LLAMA3_70B = [("qkv", 8192, 10240), ("o_proj", 8192, 8192), ("gate_up", 8192, 57344), ("down", 28672, 8192)]
