"""One layer's output columns sharded over the ranks of a ``torch.distributed`` group (one process per GPU).

The fused operator Y = X dequant(W_Q) + X W_O (Eq. 1) has no exchange step of its own: every output column depends on
its own column of the weights only.  A layer too large or too slow for one GPU is therefore cut by output columns:
rank r packs and keeps columns [n0_r, n1_r) (whole column tiles), every rank gets the same X, computes its slice of Y
with the fused call, and one all-gather puts Y together.  That all-gather is the only collective; it moves
M x N BF16 values, a tiny fraction of the weight bytes each rank streams.

This module is host logic only: the per-rank compute is the library's fused call (``binding``), the collective is
``torch.distributed`` (NCCL on GPUs).  ``compute`` can be replaced, which is how the sharding and gathering arithmetic
is tested with gloo ranks on CPU.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

COLUMN_TILE = 256          # shards are whole column tiles of the packed format


def shard_columns(N: int, world: int, align: int = COLUMN_TILE) -> list[tuple[int, int]]:
    """Contiguous column ranges, one per rank, each a multiple of ``align`` wide, widths differing by at most one
    block of ``align`` (the first ranks take the longer ones).  A rank may get an empty range when there are fewer
    blocks than ranks."""
    if N % align != 0:
        raise ValueError(f"N = {N} is not a multiple of {align}")
    blocks = N // align
    base, extra = divmod(blocks, world)
    out, n0 = [], 0
    for r in range(world):
        w = (base + (1 if r < extra else 0)) * align
        out.append((n0, n0 + w))
        n0 += w
    return out


def shard_outliers(coo_k, coo_n, coo_v, n0: int, n1: int):
    """The COO entries of columns [n0, n1), with columns counted from n0."""
    coo_n = np.asarray(coo_n)
    sel = (coo_n >= n0) & (coo_n < n1)
    return np.asarray(coo_k)[sel], (coo_n[sel] - n0).astype(np.uint32), np.asarray(coo_v)[sel]


@dataclass
class Shard:
    rank: int
    world: int
    n0: int
    n1: int

    @property
    def width(self) -> int:
        return self.n1 - self.n0


class ShardedLayer:
    """Rank-local part of an N-sharded layer.

    ``compute(X) -> Y_local`` returns this rank's (M, width) slice; the default packs the slice with the library
    and runs the fused kernel on the current CUDA device (and raises if there is none: no CPU fallback).
    ``forward`` gathers the slices of all ranks into the full (M, N) result on every rank.
    """

    def __init__(self, W: np.ndarray, mask: np.ndarray | None, coo_k, coo_n, coo_v, group_size: int, rank: int,
                 world: int, compute=None, process_group=None):
        K, N = W.shape
        self.K, self.N = K, N
        self.ranges = shard_columns(N, world)
        n0, n1 = self.ranges[rank]
        self.shard = Shard(rank, world, n0, n1)
        self.max_width = max(b - a for a, b in self.ranges)
        self.process_group = process_group
        self._compute = compute
        self._local = None
        if compute is None and n1 > n0:
            self._local = _LocalFused(np.ascontiguousarray(W[:, n0:n1]),
                                      None if mask is None else np.ascontiguousarray(mask[:, n0:n1]),
                                      *shard_outliers(coo_k, coo_n, coo_v, n0, n1), group_size)

    def local(self, X):
        """This rank's slice of Y, shape (M, width)."""
        if self._compute is not None:
            return self._compute(X, self.shard)
        if self.shard.width == 0:
            import torch
            return torch.empty((X.shape[0], 0), dtype=torch.int16, device=X.device)
        return self._local(X)

    def forward(self, X):
        """Full Y (M, N) on every rank: local slice, then one all-gather (slices padded to the widest shard)."""
        import torch
        import torch.distributed as dist
        y = self.local(X)
        M = y.shape[0]
        if self.shard.world == 1:
            return y
        padded = torch.zeros((M, self.max_width), dtype=y.dtype, device=y.device)
        padded[:, : self.shard.width] = y
        gathered = [torch.empty_like(padded) for _ in range(self.shard.world)]
        dist.all_gather(gathered, padded, group=self.process_group)
        out = torch.empty((M, self.N), dtype=y.dtype, device=y.device)
        for r, (a, b) in enumerate(self.ranges):
            out[:, a:b] = gathered[r][:, : b - a]
        return out


class _LocalFused:
    """The library's fused call on one shard (device arrays are uploaded once)."""

    def __init__(self, W, mask, coo_k, coo_n, coo_v, group_size):
        import torch
        from . import binding as fq
        if not torch.cuda.is_available():
            raise RuntimeError("the fused kernels need a CUDA device: there is no CPU fallback")
        K, N = W.shape
        self.fq = fq
        self.L = fq.fq_get_layout(K, N, group_size)
        wq, scale, zero = fq.fq_pack_int4(self.L, W, mask)
        indptr, info, packed = fq.fq_encode_tilecoo(self.L, coo_k, coo_n, coo_v)
        if packed.shape[0] == 0:
            packed = np.zeros((8, 16), dtype=np.uint8)

        def up(a):
            a = np.ascontiguousarray(a)
            a = a.view(np.int16) if a.dtype == np.uint16 else (a.view(np.int32) if a.dtype == np.uint32 else a)
            return torch.from_numpy(a).cuda()

        self.d = dict(wq=up(wq), scale=up(scale), zero=up(zero), indptr=up(indptr), info=up(info), packed=up(packed))
        self.ws = torch.zeros(fq.fq_workspace_bytes(self.L, fq.FQ_MAX_M), dtype=torch.uint8, device="cuda")
        self.N = N

    def __call__(self, X):
        import torch
        M = X.shape[0]
        Y = torch.empty((M, self.N), dtype=torch.int16, device=X.device)
        d = self.d
        self.fq.fq_fused_w4a16_outlier_gemm(self.L, X, M, d["wq"], d["scale"], d["zero"], d["indptr"], d["info"],
                                            d["packed"], Y, self.ws)
        return Y
