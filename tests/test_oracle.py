"""Pins of the CPU oracle against things other than itself: a hand-worked
example, closed forms, invariants, brute force with numpy/torch routines, and
special cases that reduce to textbook operations.  CPU only."""
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits_torch(a: np.ndarray) -> np.ndarray:
    """binary32 -> BF16 bit patterns through torch's own conversion."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# ------------------------------------------------------------------ BF16

def test_bf16_conversion_matches_torch():
    rng = np.random.default_rng(1)
    a = np.concatenate([
        rng.standard_normal(20000).astype(np.float32),
        (rng.standard_normal(2000) * 1e-30).astype(np.float32),
        (rng.standard_normal(2000) * 1e30).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 0.1, 1.00390625, 1.01171875, 3.3895314e38, np.inf, -np.inf],
                 dtype=np.float32),
    ])
    want = bf16_bits_torch(a)
    got = np.array([oracle.f32_to_bf16(float(v)) for v in a], dtype=np.uint16)
    assert np.array_equal(got, want)
    back = np.array([oracle.bf16_to_f32(int(b)) for b in want[:5000]], dtype=np.float32)
    assert np.array_equal(back.view(np.uint32), (want[:5000].astype(np.uint32) << 16))


def test_bf16_ties_round_to_even():
    # 1 + 2^-8 is exactly half way between 1 and 1 + 2^-7: goes to even (1.0)
    assert oracle.f32_to_bf16(1.00390625) == 0x3F80
    # 1 + 3 * 2^-8 is half way between 1 + 2^-7 and 1 + 2^-6: goes to even (1 + 2^-6)
    assert oracle.f32_to_bf16(1.01171875) == 0x3F82


# ------------------------------------------------------------- quantiser

def test_quantiser_hand_worked_example():
    rows, tail = [], None
    with open(os.path.join(GOLDEN, "toy_group_quant.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            parts = line.split()
            if parts[0].startswith("0x"):
                tail = (int(parts[0], 16), int(parts[1]))
            else:
                rows.append((float(parts[0]), int(parts[1]), float(parts[2])))
    W = np.array([[r[0]] for r in rows], dtype=np.float32)
    q, s, z = oracle.quantize(W, None, g=4)
    assert int(s[0, 0]) == tail[0]
    assert bf16_to_f64(z)[0, 0] == tail[1]
    assert [int(v) for v in q[:, 0]] == [r[1] for r in rows]
    What = oracle.dequant(q, s, z, 4)
    assert np.array_equal(What[:, 0], np.array([r[2] for r in rows]))


def test_quantiser_clamps_codes():
    # wmin = -0.4375, wmax = 1.4375: s = 1.875 / 15 = 0.125 (exact in BF16),
    # z = round(3.5) = 4 and round(11.5) = 12 under round-half-to-even, so Eq. 2 as
    # printed would give the code 16 for wmax; the 4-bit range needs a clamp.
    W = np.array([[-0.4375], [1.4375], [0.0], [0.05]], dtype=np.float32)
    q, s, z = oracle.quantize(W, None, g=4)
    assert int(s[0, 0]) == 0x3E00
    assert bf16_to_f64(z)[0, 0] == 4.0
    assert [int(v) for v in q[:, 0]] == [0, 15, 4, 4]


def _random_layer(K, N, g, density, seed):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((K, N)) * 0.02).astype(np.float32)
    mask = (rng.random((K, N)) < density).astype(np.uint8)
    vals = (rng.uniform(6, 20, size=(K, N)) * 0.02 * rng.choice([-1.0, 1.0], size=(K, N))).astype(np.float32)
    vb = bf16_bits_torch(vals)
    W = np.where(mask == 1, (vb.astype(np.uint32) << 16).view(np.float32), W)
    kk, nn = np.nonzero(mask)
    return W, mask, kk.astype(np.uint32), nn.astype(np.uint32), vb[kk, nn]


@pytest.mark.parametrize("g", [64, 128])
def test_quantiser_invariants(g):
    K, N = 256, 96
    W, mask, ck, cn, cv = _random_layer(K, N, g, 0.02, seed=7)
    q, s, z = oracle.quantize(W, mask, g)
    sf = bf16_to_f64(s)
    zf = bf16_to_f64(z)
    assert q.max() <= 15 and zf.max() <= 15 and zf.min() >= 0
    assert np.array_equal(zf, np.rint(zf))
    What = oracle.dequant(q, s, z, g)
    srep = np.repeat(sf, g, axis=0)
    inl = mask == 0
    # every non-outlier weight lies inside its group's [wmin, wmax], hence within s/2 (+ slack
    # of one binary32 ulp of the quotient) of a representable level unless clamping bites
    err = np.abs(W.astype(np.float64) - What)
    zrep = np.repeat(zf, g, axis=0)
    clamped = ((q == 0) | (q == 15)) & inl
    assert np.all(err[inl & ~clamped] <= srep[inl & ~clamped] * (0.5 + 1e-6))
    assert np.all(err[clamped] <= srep[clamped] * 1.0 + 1e-12)
    # an outlier slot dequantises to exactly zero
    assert np.all(What[mask == 1] == 0.0)
    assert np.array_equal(q[mask == 1], zrep[mask == 1].astype(np.uint8))
    # exact zero is always representable
    assert np.all((q.astype(np.float64) - zrep) * srep == What)


def test_quantiser_idempotent_on_its_own_output():
    K, N, g = 128, 40, 64
    W, mask, *_ = _random_layer(K, N, g, 0.0, seed=3)
    q, s, z = oracle.quantize(W, None, g)
    What = oracle.dequant(q, s, z, g).astype(np.float32)
    # re-quantising the reconstruction with the group's own (s, z) returns the same codes
    sf = np.repeat(bf16_to_f64(s), g, axis=0).astype(np.float32)
    zf = np.repeat(bf16_to_f64(z), g, axis=0)
    q2 = np.clip(np.rint(What / sf) + zf, 0, 15).astype(np.uint8)
    assert np.array_equal(q2, q)


def test_quantiser_whole_column_group_is_textbook_minmax():
    # g = K, no outliers: per-column asymmetric min-max quantisation, written with torch ops
    K, N = 64, 33
    rng = np.random.default_rng(11)
    W = (rng.standard_normal((K, N)) * 0.05 + 0.01).astype(np.float32)
    q, s, z = oracle.quantize(W, None, g=K)
    t = torch.from_numpy(W)
    wmin = torch.clamp(t.min(dim=0).values, max=0.0)
    wmax = torch.clamp(t.max(dim=0).values, min=0.0)
    sc = ((wmax - wmin) / 15.0).to(torch.bfloat16).to(torch.float32)
    zz = torch.clamp(torch.round(-wmin / sc), 0, 15)
    qq = torch.clamp(torch.round(t / sc) + zz, 0, 15).to(torch.uint8)
    assert np.array_equal(q, qq.numpy())
    assert np.array_equal(s[0], bf16_bits_torch(sc.numpy()))
    assert np.array_equal(bf16_to_f64(z)[0], zz.numpy().astype(np.float64))


def test_quantiser_degenerate_groups():
    K, N, g = 128, 4, 64
    W = np.zeros((K, N), dtype=np.float32)
    mask = np.zeros((K, N), dtype=np.uint8)
    W[:64, 1] = 0.3           # all members of group 0 / column 1 are outliers
    mask[:64, 1] = 1
    W[64:, 2] = 0.25          # one-sided group: the range is widened to contain 0
    q, s, z = oracle.quantize(W, mask, g)
    assert int(s[0, 0]) == 0x3F80 and int(z[0, 0]) == 0 and q[:64, 0].max() == 0
    assert int(s[0, 1]) == 0x3F80 and int(z[0, 1]) == 0 and q[:64, 1].max() == 0
    assert bf16_to_f64(z)[1, 2] == 0.0 and np.all(q[64:, 2] == 15)


# ---------------------------------------------------------------- result

@pytest.mark.parametrize("M,K,N,g,density", [(3, 128, 40, 64, 0.03), (5, 256, 24, 128, 0.1), (1, 64, 7, 64, 0.5)])
def test_matmul_equals_dense_brute_force(M, K, N, g, density):
    W, mask, ck, cn, cv = _random_layer(K, N, g, density, seed=K + N)
    q, s, z = oracle.quantize(W, mask, g)
    rng = np.random.default_rng(5)
    X = bf16_bits_torch(rng.standard_normal((M, K)).astype(np.float32))
    Y = oracle.fused_matmul(X, q, s, z, g, ck, cn, cv)
    # materialise W^ + W_O with numpy only and use the library matmul
    sf = np.repeat(bf16_to_f64(s), g, axis=0)
    zf = np.repeat(bf16_to_f64(z), g, axis=0)
    Wrec = sf * (q.astype(np.float64) - zf)
    WO = np.zeros((K, N))
    WO[ck, cn] = bf16_to_f64(cv)
    ref = bf16_to_f64(X) @ (Wrec + WO)
    assert np.max(np.abs(Y - ref)) <= 1e-12 * np.max(np.abs(ref))
    # a transposed operand, a dropped sparse term or a wrong sign would not survive this
    ref_dense_only = bf16_to_f64(X) @ Wrec
    assert np.max(np.abs(Y - ref_dense_only)) > 1e-6


def test_matmul_without_outliers_is_the_dequant_gemm_bit_for_bit():
    M, K, N, g = 4, 256, 32, 128
    W, *_ = _random_layer(K, N, g, 0.0, seed=21)
    q, s, z = oracle.quantize(W, None, g)
    X = bf16_bits_torch(np.random.default_rng(2).standard_normal((M, K)).astype(np.float32))
    empty = np.zeros(0, dtype=np.uint32)
    Y = oracle.fused_matmul(X, q, s, z, g, empty, empty, np.zeros(0, dtype=np.uint16))
    What = oracle.dequant(q, s, z, g)
    Xf = bf16_to_f64(X)
    ref = np.zeros((M, N))
    for k in range(K):                      # same ascending-k order, one product at a time
        ref += Xf[:, k:k + 1] * What[k:k + 1, :]
    assert np.array_equal(Y, ref)


def test_identity_activations_return_the_reconstructed_weights():
    K, N, g = 128, 48, 64
    W, mask, ck, cn, cv = _random_layer(K, N, g, 0.05, seed=9)
    q, s, z = oracle.quantize(W, mask, g)
    X = bf16_bits_torch(np.eye(K, dtype=np.float32))
    Y = oracle.fused_matmul(X, q, s, z, g, ck, cn, cv)
    What = oracle.dequant(q, s, z, g)
    WO = np.zeros((K, N))
    WO[ck, cn] = bf16_to_f64(cv)
    assert np.array_equal(Y, What + WO)
    # and at outlier positions that is the BF16 outlier itself
    assert np.array_equal(Y[ck, cn], bf16_to_f64(cv))


def test_constant_codes_closed_form():
    # q == c everywhere, X == 1: Y = K * s * (c - z)
    K, N, g, c = 256, 5, 128, 11
    q = np.full((K, N), c, dtype=np.uint8)
    s = np.full((K // g, N), 0x3E00, dtype=np.uint16)       # 0.125
    z = np.full((K // g, N), 0x4040, dtype=np.uint16)       # 3.0
    X = np.full((2, K), 0x3F80, dtype=np.uint16)            # 1.0
    e32 = np.zeros(0, dtype=np.uint32)
    Y = oracle.fused_matmul(X, q, s, z, g, e32, e32, np.zeros(0, dtype=np.uint16))
    assert np.all(Y == K * 0.125 * (c - 3))
    q[:] = 3
    Y = oracle.fused_matmul(X, q, s, z, g, e32, e32, np.zeros(0, dtype=np.uint16))
    assert np.all(Y == 0.0)


def test_column_subset_matches_full_result():
    M, K, N, g = 3, 128, 64, 64
    W, mask, ck, cn, cv = _random_layer(K, N, g, 0.04, seed=13)
    q, s, z = oracle.quantize(W, mask, g)
    X = bf16_bits_torch(np.random.default_rng(4).standard_normal((M, K)).astype(np.float32))
    Y, Yabs = oracle.fused_matmul(X, q, s, z, g, ck, cn, cv, want_abs=True)
    cols = np.array([63, 0, 17, 5], dtype=np.uint32)
    Ys, Ysabs = oracle.fused_matmul(X, q, s, z, g, ck, cn, cv, cols=cols, want_abs=True)
    assert np.array_equal(Ys, Y[:, cols]) and np.array_equal(Ysabs, Yabs[:, cols])
    assert np.all(Yabs >= np.abs(Y))


# ------------------------------------------------------- format decoders

def test_decode_wq_against_a_direct_packer():
    # pack by walking every (row, column) and computing where the format puts it
    K, N, BN = 256, 64, 32
    rng = np.random.default_rng(17)
    q = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    words = np.zeros(K * N // 8, dtype=np.uint32)
    KT = K // 128
    for row in range(K):
        kt, kr = divmod(row, 128)
        j, r32 = divmod(kr, 32)
        w, r8 = divmod(r32, 8)
        i, h = divmod(r8, 2)
        nib = i + 4 * h
        for col in range(N):
            tn, t = divmod(col, BN)
            idx = (tn * KT + kt) * 16 * BN + (j * BN + t) * 4 + w
            words[idx] |= np.uint32(int(q[row, col]) << (4 * nib))
    assert np.array_equal(oracle.decode_wq(words, K, N, BN), q)


def test_decode_tilecoo_hand_built():
    # K = 128, N = 64, BN = 32 -> 2 tiles of 8 buckets; bucket b holds the tile columns b + 8 j
    K, N, BN, NB = 128, 64, 32, 8
    slots = np.zeros((4, 4), dtype=np.uint32)

    def put(p, slot, k, j, bits):
        slots[p, slot] = (bits << 16) | (j << 3) | (k << 5)

    # tile 0, bucket 1 (columns 1, 9, 17, 25): two column-slotted packets
    put(0, 0, 5, 0, 0x3F80); put(0, 1, 0, 1, 0); put(0, 2, 127, 2, 0xBF80); put(0, 3, 0, 3, 0)
    put(1, 0, 9, 0, 0x4000); put(1, 1, 0, 1, 0); put(1, 2, 0, 2, 0); put(1, 3, 0, 3, 0)
    # tile 1, bucket 7 (columns 7, 15, 23, 31): one column-slotted packet and a tail packet whose
    # slots name any column; its last slot is all-zero padding
    put(2, 0, 0, 0, 0); put(2, 1, 0, 1, 0); put(2, 2, 0, 2, 0); put(2, 3, 3, 3, 0x3E00)
    put(3, 0, 10, 3, 0x4100); put(3, 1, 11, 3, 0x4101); put(3, 2, 11, 0, 0x4102)
    indptr = np.array([0, 2, 4], dtype=np.uint32)
    info = np.zeros(2 * NB, dtype=np.uint32)
    info[1] = 0 | (2 << 16)
    info[2:8] = 2                            # empty buckets after bucket 1
    info[NB + 7] = 0 | (1 << 16) | (1 << 24)
    packets = slots.view(np.uint8).reshape(4, 16)
    k, n, v, b = oracle.decode_tilecoo(indptr, info, packets, K, N, BN, NB)
    got = sorted(zip(k.tolist(), n.tolist(), v.tolist(), b.tolist()))
    want = sorted([(5, 1, 0x3F80, 1), (127, 17, 0xBF80, 1), (9, 1, 0x4000, 1), (3, 32 + 31, 0x3E00, NB + 7),
                   (10, 32 + 31, 0x4100, NB + 7), (11, 32 + 31, 0x4101, NB + 7), (11, 32 + 7, 0x4102, NB + 7)])
    assert got == want
    bad = info.copy()
    bad[NB + 7] = 0 | (1 << 16) | (2 << 24)  # bucket runs past its tile
    with pytest.raises(ValueError):
        oracle.decode_tilecoo(indptr, bad, packets, K, N, BN, NB)
    wrong = slots.copy()
    wrong[0, 1] = (0x3F80 << 16) | (2 << 3)  # a column-slotted slot that names another column
    with pytest.raises(ValueError):
        oracle.decode_tilecoo(indptr, info, wrong.view(np.uint8).reshape(4, 16), K, N, BN, NB)
    stray = slots.copy()
    stray[3, 0] |= 1                         # a bit outside the fields
    with pytest.raises(ValueError):
        oracle.decode_tilecoo(indptr, info, stray.view(np.uint8).reshape(4, 16), K, N, BN, NB)


def test_binary16_conversion_matches_numpy_on_every_pattern_and_enters_the_matmul():
    """The oracle's IEEE binary16 reader (outlier values of the second type in Table 1) against numpy's float16 for
    all 65536 patterns, and Eq. 1 with binary16 outliers against a dense numpy matmul."""
    import ctypes
    lib = oracle.lib()
    lib.orc_f16_to_f64.restype = ctypes.c_double
    lib.orc_f16_to_f64.argtypes = [ctypes.c_uint16]
    pats = np.arange(65536, dtype=np.uint16)
    want = pats.view(np.float16).astype(np.float64)
    got = np.array([lib.orc_f16_to_f64(int(p)) for p in pats])
    assert np.array_equal(np.isnan(got), np.isnan(want))
    ok = ~np.isnan(want)
    assert np.array_equal(got[ok], want[ok]) and np.array_equal(np.signbit(got[ok]), np.signbit(want[ok]))
    # Eq. 1: zero dense part (all codes equal the zero-point), outliers as binary16
    K, N, M, g = 128, 64, 3, 128
    rng = np.random.default_rng(11)
    q = np.full((K, N), 5, dtype=np.uint8)
    s = np.full((K // g, N), 0x3F80, dtype=np.uint16)            # scale 1
    z = np.full((K // g, N), 0x40A0, dtype=np.uint16)            # zero-point 5
    nnz = 300
    pos = rng.choice(K * N, size=nnz, replace=False)
    kk, nn = (pos // N).astype(np.uint32), (pos % N).astype(np.uint32)
    vals = rng.normal(0, 1, size=nnz).astype(np.float16)
    Xf = rng.normal(0, 1, size=(M, K)).astype(np.float32)
    Xb = (Xf.view(np.uint32) >> 16).astype(np.uint16)
    Xd = (Xb.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    Wd = np.zeros((K, N), dtype=np.float64)
    Wd[kk, nn] = vals.astype(np.float64)
    Y = oracle.fused_matmul(Xb, q, s, z, g, kk, nn, vals.view(np.uint16), value_type=1)
    assert np.allclose(Y, Xd @ Wd, rtol=0, atol=1e-12)
    # the same bits read as BF16 are other numbers: the type must matter
    Yb = oracle.fused_matmul(Xb, q, s, z, g, kk, nn, vals.view(np.uint16), value_type=0)
    assert not np.allclose(Yb, Y, rtol=1e-3, atol=1e-3)


def _pad_case(seed, K=256, N=256, density=0.02):
    rng = np.random.default_rng(seed)
    W = rng.normal(0, 0.02, size=(K, N)).astype(np.float32)
    mask = (rng.random((K, N)) < density).astype(np.uint8)
    W = np.where(mask == 1, (rng.uniform(0.12, 0.4, size=(K, N)) * rng.choice([-1, 1], size=(K, N))).astype(np.float32), W)
    return W, mask


def test_pad_slot_repurposing_worked_example():
    """Section 3.2.1's remark, on a tile small enough to check by eye.  One tile of 128 x 128, groups of 128.
    Column 0 has two outliers, columns 8, 16 and 24 (the other three columns of bucket 0) have none: the bucket is
    two packets deep and each of those three columns has two padding slots.  Every weight of column 8 sits
    exactly on the quantisation grid except rows 5 and 77; column 16 is all zero; column 24 has three off-grid
    weights.  Expected: column 8 gains rows 5 and 77, column 16 nothing (no weight with an error), column 24 its two
    worst rows; nothing else changes."""
    K = N = 128
    W = np.zeros((K, N), dtype=np.float32)
    mask = np.zeros((K, N), dtype=np.uint8)
    W[3, 0], W[90, 0] = 0.3, -0.25
    mask[3, 0] = mask[90, 0] = 1
    W[10, 0] = 0.015                                      # a plain weight of column 0: range [0, 0.015]
    # column 8: range exactly [-0.75, 0.75], scale 0.1 (BF16 of 0.1 = 0.10009765625), values on the grid s*(q-z)
    s8 = float(np.float32(np.uint32(0x3DCD << 16).view(np.float32)))
    W[0, 8], W[1, 8] = np.float32(-7 * s8), np.float32(8 * s8)          # z = 7
    for r in range(2, 128):
        W[r, 8] = np.float32(((r % 15) - 7) * s8)
    W[5, 8] = np.float32(2.4 * s8)                        # error 0.4 s
    W[77, 8] = np.float32(-3.3 * s8)                      # error 0.3 s
    # column 24: scale 0x3CA4 = 0.02001953125, range exactly [-7 s, 8 s]; three off-grid weights with errors
    # 0.009, 0.006, 0.003
    s24 = float(np.uint32(0x3CA4 << 16).view(np.float32))
    W[0, 24], W[1, 24] = np.float32(-7 * s24), np.float32(8 * s24)
    W[40, 24] = np.float32(2 * s24 + 0.009)
    W[41, 24] = np.float32(-3 * s24 - 0.006)
    W[42, 24] = np.float32(1 * s24 + 0.003)
    out = oracle.repurpose_pads(W, mask, 128, 128)
    q, s, z = oracle.quantize(W, mask, 128)
    assert s[0, 8] == 0x3DCD and oracle.bf16_to_f32(int(z[0, 8])) == 7.0
    assert s[0, 24] == 0x3CA4 and oracle.bf16_to_f32(int(z[0, 24])) == 7.0
    added = np.argwhere((out == 1) & (mask == 0))
    got = {(int(r), int(c)) for r, c in added}
    err24 = np.abs(W[:, 24].astype(np.float64) - oracle.dequant(q, s, z, 128)[:, 24])
    worst24 = set(np.argsort(-err24, kind="stable")[:2].tolist())
    assert worst24 == {40, 41}
    assert got == {(5, 8), (77, 8), (40, 24), (41, 24)}
    assert np.array_equal(out[mask == 1], mask[mask == 1])


@pytest.mark.parametrize("seed,BN", [(1, 128), (2, 256)])
def test_pad_slot_repurposing_invariants(seed, BN):
    """What the definition fixes, checked with code of its own: per (tile, column) exactly depth - count weights
    are added where that many candidates exist; they are the largest quantisation errors of the column inside the
    tile; and the matrix reconstructed under the new mask is closer to W."""
    K, N, g = 256, 256, 128
    W, mask = _pad_case(seed, K, N)
    out = oracle.repurpose_pads(W, mask, g, BN)
    assert np.all(out[mask == 1] == 1)
    q, s, z = oracle.quantize(W, mask, g)
    err = np.abs(W.astype(np.float64) - oracle.dequant(q, s, z, g))
    for tn in range(N // BN):
        for kt in range(K // 128):
            rows = slice(kt * 128, kt * 128 + 128)
            cnt = mask[rows, tn * BN:(tn + 1) * BN].sum(axis=0).astype(int)
            for b in range(BN // 4):
                cols = [32 * (b // 8) + b % 8 + 8 * j for j in range(4)]
                depth = max(cnt[c] for c in cols)
                for c in cols:
                    n = tn * BN + c
                    new = (out[rows, n] == 1) & (mask[rows, n] == 0)
                    assert new.sum() == depth - cnt[c]
                    if new.any():
                        rest = (out[rows, n] == 0)
                        assert err[rows, n][new].min() >= err[rows, n][rest].max()
    def recon_error(m):
        q2, s2, z2 = oracle.quantize(W, m, g)
        What = oracle.dequant(q2, s2, z2, g)
        bf = ((W.view(np.uint32) + 0x7fff + ((W.view(np.uint32) >> 16) & 1)) & 0xffff0000).view(np.float32).astype(np.float64)
        R = np.where(m == 1, bf, What)
        return np.linalg.norm(W.astype(np.float64) - R)
    assert recon_error(out) < recon_error(mask)

