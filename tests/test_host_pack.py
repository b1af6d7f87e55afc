"""Host half of the library (packer, Tile-COO encoder / decoder / validator) against the oracle
and against the invariants the paper states.  CPU only: no kernel is launched here."""
import os
import re

import numpy as np
import pytest

import oracle
from paper_2608_15531_b200 import binding as fq
from paper_2608_15531_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "fq.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = sorted(set(re.findall(r"\b(fq_[a-z0-9_]+)\s*\(", hdr)))
    assert len(declared) >= 15
    lib = fq.lib()
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in fq.h but not exported"
    assert sorted(fq.EXPORTS) == declared


def test_layout_defaults_and_errors():
    L = fq.fq_get_layout(4096, 4096, 128)
    assert (L.BK, L.BN, L.buckets_per_tile, L.coo_unit_bytes) == (128, 256, 64, 16)
    assert fq.fq_get_layout(4096, 4224, 64).BN == 128
    for bad in [(4096, 4096, 32), (4000, 4096, 128), (4096, 4100, 128)]:
        with pytest.raises(fq.FqError) as e:
            fq.fq_get_layout(*bad)
        assert e.value.code == fq.FQ_ERR_UNSUPPORTED_SHAPE
    with pytest.raises(fq.FqError):
        fq.fq_get_layout(4096, 4096, 128, bn_hint=64)
    with pytest.raises(fq.FqError):
        fq.fq_get_layout(4096, 4096, 128, nb_hint=48)
    with pytest.raises(fq.FqError) as e:
        fq.fq_workspace_bytes(L, 129)
    assert e.value.code == fq.FQ_ERR_INVALID_ARG
    assert fq.fq_workspace_bytes(L, 1) > 0


@pytest.mark.parametrize("K,N,g,BN,layout", [(256, 512, 128, 256, "mixed"), (384, 384, 64, 128, "uniform"),
                                              (512, 768, 128, 256, "clustered")])
def test_pack_round_trips_against_the_oracle(K, N, g, BN, layout):
    Lr = synth.layer(synth.tensor_seed(0, K + N), K, N, density=0.02, layout=layout)
    L = fq.fq_get_layout(K, N, g, bn_hint=BN)
    wq, s, z = fq.fq_pack_int4(L, Lr.W, Lr.mask)
    q_o, s_o, z_o = oracle.quantize(Lr.W, Lr.mask, g)
    assert wq.nbytes == K * N // 2 and s.shape == (K // g, N)
    assert np.array_equal(s, s_o) and np.array_equal(z, z_o)
    assert np.array_equal(oracle.decode_wq(wq, K, N, BN), q_o)       # oracle's own reader of the format
    assert np.array_equal(fq.fq_unpack_int4(L, wq), q_o)             # library's inverse
    # without a mask the outlier magnitudes widen the group ranges: results must differ
    wq2, s2, _ = fq.fq_pack_int4(L, Lr.W, None)
    assert not np.array_equal(s2, s)


def test_pack_degenerate_and_one_sided_groups():
    K, N, g = 128, 128, 64
    W = np.zeros((K, N), dtype=np.float32)
    mask = np.zeros((K, N), dtype=np.uint8)
    W[:64, 1] = 0.3
    mask[:64, 1] = 1
    W[64:, 2] = 0.25
    W[:, 3] = -0.125
    L = fq.fq_get_layout(K, N, g)
    wq, s, z = fq.fq_pack_int4(L, W, mask)
    q_o, s_o, z_o = oracle.quantize(W, mask, g)
    assert np.array_equal(s, s_o) and np.array_equal(z, z_o)
    assert np.array_equal(fq.fq_unpack_int4(L, wq), q_o)


def _as_set(k, n, v):
    return set(zip(k.tolist(), n.tolist(), v.tolist()))


def _bank_conflict_cycles(bk, bb, order_pos, NB):
    """Shared-memory passes of the sparse lanes' activation reads (32-byte FP32 rows, so rows k and
    k + 4 share banks): lanes (= buckets) are served eight at a time; at entry position i the passes
    needed are the largest number of different rows falling in one bank group (k mod 4)."""
    cycles = 0
    per_bucket = {}
    for k, b, pos in zip(bk, bb, order_pos):
        per_bucket.setdefault(int(b), {})[int(pos)] = int(k)
    depth = max((len(v) for v in per_bucket.values()), default=0)
    for q0 in range(0, NB, 8):
        for i in range(depth):
            rows = {per_bucket[b][i] for b in range(q0, q0 + 8) if b in per_bucket and i in per_bucket[b]}
            groups = {}
            for k in rows:
                groups[k % 4] = groups.get(k % 4, 0) + 1
            cycles += max(groups.values(), default=0)
    return cycles


@pytest.mark.parametrize("layout,density,NB", [("uniform", 0.01, 32), ("mixed", 0.02, 64), ("clustered", 0.05, 128)])
def test_tilecoo_encode_invariants(layout, density, NB):
    K, N, BN = 512, 1024, 256
    Lr = synth.layer(synth.tensor_seed(3, NB), K, N, density=density, layout=layout)
    L = fq.fq_get_layout(K, N, 128, bn_hint=BN, nb_hint=NB)
    n_ip, n_bi, n_pk, mx = fq.fq_encode_tilecoo_sizes(L, Lr.coo_k, Lr.coo_n, Lr.coo_v)
    indptr, info, packed = fq.fq_encode_tilecoo(L, Lr.coo_k, Lr.coo_n, Lr.coo_v)
    ntile = (K // 128) * (N // BN)
    # array sizes and storage formula (Table 1 and the storage analysis), padding bounded per bucket
    assert n_ip == ntile + 1 == indptr.size and n_bi == ntile * NB == info.size and n_pk == packed.shape[0]
    assert L.max_tile_packets == mx == int(np.diff(indptr).max())
    assert indptr[0] == 0 and np.all(np.diff(indptr.astype(np.int64)) >= 0) and indptr[-1] == n_pk
    assert 4 * Lr.nnz <= 16 * n_pk <= 16 * Lr.nnz          # every packet carries at least one outlier
    # decoded set == input set, by the oracle's reader and by the library's
    want = _as_set(Lr.coo_k, Lr.coo_n, Lr.coo_v)
    k, n, v, b = oracle.decode_tilecoo(indptr, info, packed, K, N, BN, NB)
    assert len(k) == Lr.nnz and _as_set(k, n, v) == want
    k2, n2, v2 = fq.fq_decode_tilecoo(L, indptr, info, packed)
    assert _as_set(k2, n2, v2) == want
    fq.fq_validate_tilecoo(L, indptr, info, packed)
    # buckets of a tile own disjoint column sets (the sparse path's conflict-free accumulation)
    tile = (n // BN) * (K // 128) + k // 128
    owner = {}
    for t_, c_, b_ in zip(tile.tolist(), n.tolist(), b.tolist()):
        assert owner.setdefault((t_, c_), b_) == b_
    # a column lives in one block of 32 buckets (column mod number of blocks) in every tile; inside a
    # block the greedy least-loaded assignment gives max bucket load <= mean load + largest column
    nblk = NB // 32
    assert np.array_equal((b % NB) // 32, (n % BN) % nblk)
    for t_ in np.unique(tile):
        sel = tile == t_
        loads = np.bincount(b[sel] - t_ * NB, minlength=NB)
        for blk in range(nblk):
            in_blk = sel & ((n % BN) % nblk == blk)
            colmax = np.bincount(n[in_blk] % BN, minlength=BN).max() if in_blk.any() else 0
            bl = loads[32 * blk:32 * blk + 32]
            assert bl.max() <= bl.sum() / 32 + colmax + 1e-9


def test_tilecoo_element_order_separates_columns_and_staggers_bank_groups():
    K, N, BN, NB = 128, 256, 256, 32
    Lr = synth.layer(77, K, N, density=0.06, layout="uniform")
    L = fq.fq_get_layout(K, N, 128, bn_hint=BN, nb_hint=NB)
    indptr, info, packed = fq.fq_encode_tilecoo(L, Lr.coo_k, Lr.coo_n, Lr.coo_v)
    k, n, v, b = oracle.decode_tilecoo(indptr, info, packed, K, N, BN, NB)   # decode keeps stored order
    pos = np.zeros(len(k), dtype=np.int64)
    seen = {}
    for i, bb in enumerate(b.tolist()):
        pos[i] = seen.get(bb, 0)
        seen[bb] = pos[i] + 1
    # rule 1: a packet is either "spread" (its outliers sit in different columns) or "stack" (four
    # outliers of one column); a stack is only formed while fewer than four columns have entries left
    raw = packed.reshape(-1, 16)
    for bb in np.unique(b):
        t_, lb = divmod(int(bb), NB)
        off, cnt = int(info[bb]) & 0xffff, int(info[bb]) >> 16
        left = {}
        for c in (n[b == bb] % BN).tolist():
            left[c] = left.get(c, 0) + 1
        for pk in raw[int(indptr[t_]) + off:int(indptr[t_]) + off + cnt]:
            vals = pk[8:].view(np.uint16)
            cols = [int(pk[4 + s_]) for s_ in range(4) if vals[s_] != 0]
            assert len(cols) >= 1
            if len(set(cols)) < len(cols):
                assert len(cols) == 4 and len(set(cols)) == 1
                assert sum(1 for v_ in left.values() if v_ > 0) < 4
            else:
                alive = sum(1 for v_ in left.values() if v_ > 0)
                assert len(cols) == min(4, alive)
            for c in cols:
                left[c] -= 1
        assert all(v_ == 0 for v_ in left.values())
    # rule 2 pays off: fewer shared-memory passes than the plain (column, row) order
    plain_pos = np.zeros(len(k), dtype=np.int64)
    for bb in np.unique(b):
        idx = np.nonzero(b == bb)[0]
        order = sorted(idx.tolist(), key=lambda i: (int(n[i]), int(k[i])))
        for p_, i in enumerate(order):
            plain_pos[i] = p_
    assert _bank_conflict_cycles(k, b, pos, NB) < _bank_conflict_cycles(k, b, plain_pos, NB)
    # a bucket that owns a single hot column cannot avoid repeats, and still round-trips
    kk = np.arange(0, 40, dtype=np.uint32)
    nn = np.full(40, 7, dtype=np.uint32)
    vv = (0x3F80 + np.arange(40)).astype(np.uint16)
    ip, bi, pk = fq.fq_encode_tilecoo(L, kk, nn, vv)
    k2, n2, v2 = fq.fq_decode_tilecoo(L, ip, bi, pk)
    assert _as_set(k2, n2, v2) == _as_set(kk, nn, vv) and pk.shape[0] == 10          # ten stacks of four


def test_tilecoo_edge_cases():
    K, N, BN, NB = 256, 512, 256, 32
    L = fq.fq_get_layout(K, N, 128, bn_hint=BN, nb_hint=NB)
    e32, e16 = np.zeros(0, dtype=np.uint32), np.zeros(0, dtype=np.uint16)
    # no outliers at all
    indptr, info, packed = fq.fq_encode_tilecoo(L, e32, e32, e16)
    assert packed.shape[0] == 0 and not indptr.any() and not info.any() and L.max_tile_packets == 0
    fq.fq_validate_tilecoo(L, indptr, info, packed)
    # a single outlier; zero-valued entries are dropped
    k = np.array([200, 5, 6], dtype=np.uint32)
    n = np.array([300, 7, 8], dtype=np.uint32)
    v = np.array([0x4000, 0x0000, 0x8000], dtype=np.uint16)
    indptr, info, packed = fq.fq_encode_tilecoo(L, k, n, v)
    assert packed.shape[0] == 1
    kk, nn, vv, _ = oracle.decode_tilecoo(indptr, info, packed, K, N, BN, NB)
    assert (kk.tolist(), nn.tolist(), vv.tolist()) == ([200], [300], [0x4000])
    # padding slots: value 0, row 0, a column byte that differs from slot to slot
    assert packed[0, :4].tolist() == [72, 0, 0, 0] and packed[0, 4:8].tolist() == [44, 254, 253, 252]
    assert packed[0, 10:].tolist() == [0] * 6
    # one completely dense tile plus a hot row and a hot column elsewhere
    kk, nn = np.meshgrid(np.arange(128, 256), np.arange(0, 256), indexing="ij")
    k = np.concatenate([kk.ravel(), np.full(256, 3), np.arange(0, 128)]).astype(np.uint32)
    n = np.concatenate([nn.ravel(), np.arange(256, 512), np.full(128, 400)]).astype(np.uint32)
    keep = np.unique(np.stack([k, n]), axis=1)
    k, n = keep[0].astype(np.uint32), keep[1].astype(np.uint32)
    v = (0x3F80 + (np.arange(k.size) % 64)).astype(np.uint16)
    indptr, info, packed = fq.fq_encode_tilecoo(L, k, n, v)
    assert L.max_tile_packets == 128 * 256 // 4
    k2, n2, v2 = fq.fq_decode_tilecoo(L, indptr, info, packed)
    assert _as_set(k2, n2, v2) == _as_set(k, n, v)
    fq.fq_validate_tilecoo(L, indptr, info, packed)
    with pytest.raises(fq.FqError) as e:
        fq.fq_encode_tilecoo(L, np.array([256], dtype=np.uint32), np.array([0], dtype=np.uint32),
                             np.array([0x4000], dtype=np.uint16))
    assert e.value.code == fq.FQ_ERR_INVALID_ARG


def test_validator_rejects_corrupted_arrays():
    K, N, BN, NB = 256, 512, 256, 32
    Lr = synth.layer(5, K, N, density=0.02, layout="mixed")
    L = fq.fq_get_layout(K, N, 128, bn_hint=BN, nb_hint=NB)
    indptr, info, packed = fq.fq_encode_tilecoo(L, Lr.coo_k, Lr.coo_n, Lr.coo_v)
    fq.fq_validate_tilecoo(L, indptr, info, packed)

    def expect_format_error(ip, bi, pk):
        with pytest.raises(fq.FqError) as e:
            fq.fq_validate_tilecoo(L, ip, bi, pk)
        assert e.value.code == fq.FQ_ERR_FORMAT

    bad = indptr.copy(); bad[2] = bad[1] - 1 if bad[1] > 0 else 2 ** 31
    expect_format_error(bad, info, packed)
    bad = indptr.copy(); bad[-1] += 1
    expect_format_error(bad, info, packed)
    bad = info.copy(); bad[0] = (bad[0] & 0xffff) | (0xffff << 16)
    expect_format_error(indptr, bad, packed)
    bad = packed.copy(); bad[0, 0] = 200                 # row index outside the 128-row tile
    expect_format_error(indptr, info, bad)
    # move one entry into a column another bucket of the same tile owns
    k, n, v, b = oracle.decode_tilecoo(indptr, info, packed, K, N, BN, NB)
    first_tile = b < NB
    cols0 = n[first_tile & (b == b[first_tile][0])] % BN
    other = n[first_tile & (b != b[first_tile][0])] % BN
    bad = packed.copy()
    off0 = int(info[int(b[first_tile][0])] & 0xffff)
    bad[off0, 4] = int(other[0])
    assert int(other[0]) not in cols0.tolist()
    expect_format_error(indptr, info, bad)
