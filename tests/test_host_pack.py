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
    L128 = fq.fq_get_layout(4096, 4224, 64)
    assert (L128.BN, L128.buckets_per_tile) == (128, 32)
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


def _bucket_of(c):
    """Bucket of a tile column: columns g, g + 8, g + 16, g + 24 of a 32-column block share a bucket."""
    return (c // 32) * 8 + c % 8


def _fields(info):
    """offset, column-slotted packets, tail packets of every bucket descriptor."""
    return info & 0xffff, (info >> 16) & 0xff, info >> 24


def _column_counts(k, n, K, N, BN):
    """Outliers per (tile, bucket, column number inside the bucket)."""
    ntile = (K // 128) * (N // BN)
    tile = (n // BN) * (K // 128) + k // 128
    c = n % BN
    cnt = np.zeros((ntile, BN // 4, 4), dtype=np.int64)
    np.add.at(cnt, (tile, _bucket_of(c), (c // 8) % 4), 1)
    return cnt


@pytest.mark.parametrize("layout,density,BN", [("uniform", 0.01, 256), ("mixed", 0.02, 256), ("clustered", 0.05, 128)])
def test_tilecoo_encode_invariants(layout, density, BN):
    K, N = 512, 1024
    NB = BN // 4
    Lr = synth.layer(synth.tensor_seed(3, BN + len(layout)), K, N, density=density, layout=layout)
    L = fq.fq_get_layout(K, N, 128, bn_hint=BN)
    assert L.buckets_per_tile == NB
    n_ip, n_bi, n_pk, mx = fq.fq_encode_tilecoo_sizes(L, Lr.coo_k, Lr.coo_n, Lr.coo_v)
    indptr, info, packed = fq.fq_encode_tilecoo(L, Lr.coo_k, Lr.coo_n, Lr.coo_v)
    ntile = (K // 128) * (N // BN)
    off, depth, tail = _fields(info)
    # array sizes and storage formula (Table 1 and the storage analysis)
    assert n_ip == ntile + 1 == indptr.size and n_bi == ntile * NB == info.size and n_pk == packed.shape[0]
    assert L.max_tile_packets == mx == int(np.diff(indptr).max())
    assert L.max_bucket_packets == int((depth + tail).max()) and L.max_tail_packets == int(tail.max())
    assert L.tilecoo_encoded == 1
    assert indptr[0] == 0 and np.all(np.diff(indptr.astype(np.int64)) >= 0) and indptr[-1] == n_pk
    assert 4 * Lr.nnz <= 16 * n_pk <= 16 * Lr.nnz          # every packet carries at least one outlier
    # decoded set == input set, by the oracle's reader and by the library's
    want = _as_set(Lr.coo_k, Lr.coo_n, Lr.coo_v)
    k, n, v, b = oracle.decode_tilecoo(indptr, info, packed, K, N, BN, NB)
    assert len(k) == Lr.nnz and _as_set(k, n, v) == want
    k2, n2, v2 = fq.fq_decode_tilecoo(L, indptr, info, packed)
    assert _as_set(k2, n2, v2) == want
    fq.fq_validate_tilecoo(L, indptr, info, packed)
    # every outlier sits in the bucket of its column, in every tile (the conflict-free accumulation of
    # the sparse path: a bucket's four columns belong to one group of four lanes)
    assert np.array_equal(b % NB, _bucket_of(n % BN))
    tile = (n // BN) * (K // 128) + k // 128
    assert np.array_equal(b // NB, tile)
    # per-column padding (Section 4.2): a bucket has as many column-slotted packets as its longest
    # column has outliers; only a column with more than 32 turns that into 4 packets and a tail
    cnt = _column_counts(Lr.coo_k.astype(np.int64), Lr.coo_n.astype(np.int64), K, N, BN).reshape(ntile * NB, 4)
    longest = cnt.max(axis=1)
    want_depth = np.where(longest > 32, 4, longest)
    want_tail = np.where(longest > 32, (np.maximum(cnt - 4, 0).sum(axis=1) + 3) // 4, 0)
    assert np.array_equal(depth, want_depth) and np.array_equal(tail, want_tail)
    if layout == "clustered":
        assert tail.any()
    else:
        assert not tail.any()
    off = off.reshape(ntile, NB)
    tot = (depth + tail).reshape(ntile, NB)
    assert np.array_equal(off[:, 1:], np.cumsum(tot, axis=1)[:, :-1]) and not off[:, 0].any()


def test_tilecoo_slots_and_order_inside_a_bucket():
    K, N, BN = 128, 256, 256
    NB = BN // 4
    Lr = synth.layer(77, K, N, density=0.03, layout="uniform")
    L = fq.fq_get_layout(K, N, 128, bn_hint=BN)
    L.slot_order = 1                                      # by row: the order this test writes out
    indptr, info, packed = fq.fq_encode_tilecoo(L, Lr.coo_k, Lr.coo_n, Lr.coo_v)
    off, depth, tail = _fields(info)
    assert not tail.any()
    slots = packed.view(np.uint32).reshape(-1, 4)
    for bb in range(NB):
        pk = slots[off[bb]:off[bb] + depth[bb]]
        # slot j of every packet names column number j, padding included
        assert np.array_equal((pk >> 3) & 3, np.tile(np.arange(4, dtype=np.uint32), (pk.shape[0], 1)))
        assert not (pk & 0x1007).any()
        for j in range(4):
            col = (bb // 8) * 32 + bb % 8 + 8 * j
            want = np.sort(Lr.coo_k[Lr.coo_n == col])
            live = (pk[:, j] >> 16) != 0
            # a column's outliers come first, by row; then only padding (value 0, row 0)
            assert live.sum() == want.size and live[:want.size].all()
            assert np.array_equal((pk[:want.size, j] >> 5) & 127, want)
            assert not (pk[want.size:, j] & 0xffffefe0).any()
    # a hot column: its first four outliers in column-slotted packets, the rest four to a packet by row
    kk = np.arange(0, 40, dtype=np.uint32)
    nn = np.full(40, 15, dtype=np.uint32)                 # column number 1 of bucket 7
    vv = (0x3F80 + np.arange(40)).astype(np.uint16)
    ip, bi, pk = fq.fq_encode_tilecoo(L, kk, nn, vv)
    k2, n2, v2 = fq.fq_decode_tilecoo(L, ip, bi, pk)
    assert _as_set(k2, n2, v2) == _as_set(kk, nn, vv) and pk.shape[0] == 4 + 9
    assert int(bi[_bucket_of(15)]) == 0 | (4 << 16) | (9 << 24)
    assert L.max_tail_packets == 9 and L.max_bucket_packets == 13
    s2 = pk.view(np.uint32).reshape(-1, 4)
    assert np.array_equal((s2[:4, 1] >> 5) & 127, np.arange(4)) and not (s2[:4, [0, 2, 3]] >> 16).any()
    assert np.array_equal((s2[4:].ravel() >> 5) & 127, np.arange(4, 40)) and np.all((s2[4:].ravel() >> 3) & 3 == 1)
    # exactly 32 in a column still has no tail
    ip, bi, pk = fq.fq_encode_tilecoo(L, kk[:32], nn[:32], vv[:32])
    assert int(bi[_bucket_of(15)]) == 0 | (32 << 16) and L.max_tail_packets == 0


def _row_read_wavefronts(L, indptr, info, packed):
    """Shared-memory wavefronts of the outlier step that reads a k-major FP32 copy of eight activation rows
    (32 B per row: rows with equal k mod 4 share banks).  One 8-byte load instruction of a warp reads slot j of
    packet d of its eight buckets; the hardware serves it half a warp at a time, i.e. four buckets' rows, and
    needs as many passes as the fullest bank group has different rows (lanes that read the same row are served
    together).  A lane group past its own list reads row 0 (padding).  Returns (wavefronts, instructions x 2
    half warps = the conflict-free minimum)."""
    NB = L.buckets_per_tile
    off, depth, _ = _fields(info)
    slots = packed.view(np.uint32).reshape(-1, 4)
    ntile = indptr.size - 1
    waves = least = 0
    for t in range(ntile):
        for s in range(NB // 8):
            dmax = int(depth[t * NB + 8 * s: t * NB + 8 * s + 8].max())
            for d in range(dmax):
                rows = np.zeros((8, 4), dtype=np.uint32)
                for gg in range(8):
                    bb = t * NB + 8 * s + gg
                    if d < depth[bb]:
                        rows[gg] = (slots[int(indptr[t]) + int(off[bb]) + d] >> 5) & 127
                for half in range(2):
                    for j in range(4):
                        distinct = np.unique(rows[4 * half: 4 * half + 4, j])
                        waves += int(np.bincount(distinct & 3, minlength=4).max())
                        least += 1
    return waves, least


@pytest.mark.parametrize("layout,density", [("uniform", 0.01), ("mixed", 0.01), ("clustered", 0.02), ("uniform", 0.03)])
def test_bank_aware_slot_order_has_fewer_conflicts_than_row_order(layout, density):
    """Section 3.2.2's element reordering, restated for this library's kernels: the default order of a column's
    outliers over its packets must decode to the same set as the row order, keep every format invariant, and
    cost the row-by-lane outlier step no more shared-memory wavefronts (clearly fewer where outliers are spread)."""
    K, N = 512, 1024
    Lr = synth.layer(91, K, N, density=density, layout=layout)
    res = {}
    for order in (0, 1):
        L = fq.fq_get_layout(K, N, 128)
        L.slot_order = order
        indptr, info, packed = fq.fq_encode_tilecoo(L, Lr.coo_k, Lr.coo_n, Lr.coo_v)
        fq.fq_validate_tilecoo(L, indptr, info, packed)
        k2, n2, v2 = fq.fq_decode_tilecoo(L, indptr, info, packed)
        assert _as_set(k2, n2, v2) == _as_set(Lr.coo_k, Lr.coo_n, Lr.coo_v)
        ko, no, vo, _ = oracle.decode_tilecoo(indptr, info, packed, L.K, L.N, L.BN, L.buckets_per_tile)
        assert _as_set(ko, no, vo) == _as_set(Lr.coo_k, Lr.coo_n, Lr.coo_v)
        res[order] = (_row_read_wavefronts(L, indptr, info, packed), info.copy(), packed.shape[0])
    (w_bank, least), info_bank, n_bank = res[0]
    (w_row, least_row), info_row, n_row = res[1]
    assert np.array_equal(info_bank, info_row) and n_bank == n_row and least == least_row   # same sizes, same descriptors
    assert w_bank <= w_row
    if layout != "clustered":
        assert (w_bank - least) < 0.8 * (w_row - least), (w_bank, w_row, least)


def test_fp16_outlier_values_round_trip_exactly():
    """Table 1's value field as IEEE binary16: the packed slots hold every binary16 number exactly (normal,
    subnormal, largest), the decoders return the same bits, and a layout of the other type rejects what it
    cannot hold."""
    K, N = 256, 512
    rng = np.random.default_rng(3)
    nnz = 4000
    pos = rng.choice(K * N, size=nnz, replace=False)
    kk, nn = (pos // N).astype(np.uint32), (pos % N).astype(np.uint32)
    vals = (rng.uniform(0.12, 0.4, size=nnz) * rng.choice([-1, 1], size=nnz)).astype(np.float16)
    vb = vals.view(np.uint16).copy()
    vb[:6] = [0x0001, 0x83ff, 0x0400, 0x7bff, 0xfbff, 0x3c01]     # subnormals, smallest normal, +-65504, 1 + 2^-10
    L = fq.fq_get_layout(K, N, 128)
    L.value_type = fq.FQ_VALUE_FP16
    indptr, info, packed = fq.fq_encode_tilecoo(L, kk, nn, vb)
    fq.fq_validate_tilecoo(L, indptr, info, packed)
    k2, n2, v2 = fq.fq_decode_tilecoo(L, indptr, info, packed)
    assert _as_set(k2, n2, v2) == _as_set(kk, nn, vb)
    ko, no, vo, _ = oracle.decode_tilecoo(indptr, info, packed, K, N, L.BN, L.buckets_per_tile, value_type=1)
    assert _as_set(ko, no, vo) == _as_set(kk, nn, vb)
    # the slot's value field is the FP32 number itself
    slots = packed.view(np.uint32).ravel()
    live = slots[(slots >> 13) != 0]
    assert sorted((live & 0xffffe000).view(np.float32).tolist()) == sorted(vb.view(np.float16).astype(np.float32).tolist())
    # these arrays are not BF16 arrays: a BF16 layout rejects them, and the oracle's BF16 reader refuses them too
    Lb = fq.fq_get_layout(K, N, 128)
    Lb.max_tile_packets, Lb.max_bucket_packets, Lb.max_tail_packets, Lb.tilecoo_encoded = \
        L.max_tile_packets, L.max_bucket_packets, L.max_tail_packets, 1
    with pytest.raises(fq.FqError) as e:
        fq.fq_validate_tilecoo(Lb, indptr, info, packed)
    assert e.value.code == fq.FQ_ERR_FORMAT
    with pytest.raises(ValueError):
        oracle.decode_tilecoo(indptr, info, packed, K, N, L.BN, L.buckets_per_tile, value_type=0)
    # and a BF16 value with eight significant bits and a large exponent is not a binary16 number
    Lb2 = fq.fq_get_layout(K, N, 128)
    ip, bi, pk = fq.fq_encode_tilecoo(Lb2, kk[:4], nn[:4], np.array([0x4780, 0x3F80, 0x0080, 0x3F81], dtype=np.uint16))
    fq.fq_validate_tilecoo(Lb2, ip, bi, pk)
    Lb2.value_type = fq.FQ_VALUE_FP16
    with pytest.raises(fq.FqError) as e:
        fq.fq_validate_tilecoo(Lb2, ip, bi, pk)          # 0x4780 = 65536 and 0x0080 = 2^-126 are out of range
    assert e.value.code == fq.FQ_ERR_FORMAT


@pytest.mark.parametrize("layout,BN,g", [("uniform", 256, 128), ("mixed", 128, 64), ("clustered", 256, 128)])
def test_pad_slot_repurposing_matches_the_oracle_and_costs_no_packets(layout, BN, g):
    """Section 3.2.1's remark on padding slots: the library picks exactly the weights the oracle picks, the packed
    outliers take exactly as many packets as before, every padding slot of a bucket without a tail is in use, and
    the reconstruction error drops."""
    K, N = 512, 512
    Lr = synth.layer(404, K, N, density=0.01, layout=layout)
    L = fq.fq_get_layout(K, N, g, bn_hint=BN)
    mask2, added = fq.fq_repurpose_pad_slots(L, Lr.W, Lr.mask)
    want = oracle.repurpose_pads(Lr.W, Lr.mask, g, BN)
    assert np.array_equal(mask2, want) and added == int(want.sum()) - int(Lr.mask.sum()) and added > 0
    ip0, bi0, pk0 = fq.fq_encode_tilecoo(L, Lr.coo_k, Lr.coo_n, Lr.coo_v)
    kk, nn = np.nonzero(mask2)
    vv = ((Lr.W[kk, nn].view(np.uint32) + 0x7fff + ((Lr.W[kk, nn].view(np.uint32) >> 16) & 1)) >> 16).astype(np.uint16)
    L2 = fq.fq_get_layout(K, N, g, bn_hint=BN)
    ip1, bi1, pk1 = fq.fq_encode_tilecoo(L2, kk.astype(np.uint32), nn.astype(np.uint32), vv)
    assert np.array_equal(ip0, ip1) and np.array_equal(bi0, bi1) and pk0.shape == pk1.shape
    off, depth, tail = _fields(bi1)
    slots = pk1.view(np.uint32).reshape(-1, 4)
    ntile = ip1.size - 1
    NB = L.buckets_per_tile
    for t in range(ntile):
        for b in range(NB):
            i = t * NB + b
            if tail[i] == 0:
                assert ((slots[ip1[t] + off[i]: ip1[t] + off[i] + depth[i]] >> 13) != 0).all()
    # the packed weights under the new mask reconstruct W more closely
    def recon_error(m, k_, n_, v_):
        q, s, z = oracle.quantize(Lr.W, m, g)
        R = oracle.dequant(q, s, z, g)
        R[k_, n_] = (v_.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        return np.linalg.norm(Lr.W.astype(np.float64) - R)
    assert recon_error(mask2, kk, nn, vv) < recon_error(Lr.mask, Lr.coo_k, Lr.coo_n, Lr.coo_v)


def test_tilecoo_edge_cases():
    K, N, BN, NB = 256, 512, 256, 64
    L = fq.fq_get_layout(K, N, 128, bn_hint=BN)
    e32, e16 = np.zeros(0, dtype=np.uint32), np.zeros(0, dtype=np.uint16)
    # no outliers at all
    assert L.tilecoo_encoded == 0
    indptr, info, packed = fq.fq_encode_tilecoo(L, e32, e32, e16)
    assert packed.shape[0] == 0 and not indptr.any() and not info.any() and L.max_tile_packets == 0 and L.tilecoo_encoded == 1
    fq.fq_validate_tilecoo(L, indptr, info, packed)
    # a single outlier; zero-valued entries are dropped
    k = np.array([200, 5, 6], dtype=np.uint32)
    n = np.array([300, 7, 8], dtype=np.uint32)
    v = np.array([0x4000, 0x0000, 0x8000], dtype=np.uint16)
    indptr, info, packed = fq.fq_encode_tilecoo(L, k, n, v)
    assert packed.shape[0] == 1
    kk, nn, vv, _ = oracle.decode_tilecoo(indptr, info, packed, K, N, BN, NB)
    assert (kk.tolist(), nn.tolist(), vv.tolist()) == ([200], [300], [0x4000])
    # column 300 = tile column 44 = column number 1 of bucket 8 + 4; the other slots are padding that
    # names their own column number
    assert packed.view(np.uint32).reshape(-1, 4)[0].tolist() == [0 << 3, (0x4000 << 16) | (1 << 3) | (72 << 5), 2 << 3, 3 << 3]
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
    K, N, BN, NB = 256, 512, 256, 64
    Lr = synth.layer(5, K, N, density=0.02, layout="mixed")
    L = fq.fq_get_layout(K, N, 128, bn_hint=BN)
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
    slots = packed.view(np.uint32).reshape(-1, 4)
    bad = slots.copy(); bad[0, 0] |= 1 << 12             # a bit outside the fields
    expect_format_error(indptr, info, bad.view(np.uint8).reshape(-1, 16))
    bad = slots.copy(); bad[0, 2] |= 1 << 2
    expect_format_error(indptr, info, bad.view(np.uint8).reshape(-1, 16))
    # a column-slotted slot that names another column of the bucket
    k, n, v, b = oracle.decode_tilecoo(indptr, info, packed, K, N, BN, NB)
    b0 = int(b[0])
    assert b0 < NB and (int(info[b0]) >> 16) & 0xff > 0
    off0 = int(info[b0] & 0xffff)
    bad = slots.copy()
    bad[off0, 1] ^= 1 << 3
    expect_format_error(indptr, info, bad.view(np.uint8).reshape(-1, 16))
    # more column-slotted packets than the format allows
    bad = info.copy(); bad[0] = (bad[0] & 0xffff) | (33 << 16)
    expect_format_error(indptr, bad, packed)
