"""Parity of the CUDA path against the CPU oracle, through the C ABI.  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_2608_15531_b200 import binding as fq
from paper_2608_15531_b200 import synth

import harness as H

pytestmark = pytest.mark.gpu


def _x(seed, M, K):
    return synth.activations(seed, M, K)


# ------------------------------------------------------------------ element-by-element, small

@pytest.mark.parametrize("K,N,g,BN,density,layout", [
    (512, 512, 128, 256, 0.01, "mixed"),       # 8 units: every CTA holds a partial piece
    (512, 768, 64, 256, 0.02, "uniform"),
    (1024, 640, 128, 128, 0.01, "mixed"),      # BN = 128 layout, ragged tile count
    (2048, 1024, 64, 128, 0.05, "clustered"),  # hot columns: long packet lists in a few buckets
    (4096, 4096, 128, 256, 0.01, "mixed"),     # configuration 1: 512 units over all SMs
    (1536, 2304, 128, 256, 0.0, "uniform"),    # no outliers at all
])
@pytest.mark.parametrize("M", [1, 3, 5, 8, 9, 16])
def test_fused_matches_oracle(K, N, g, BN, density, layout, M):
    """Every element against the oracle, twice: through the kernel the library picks for the shape (the short-job
    kernel on these small layers) and through the streaming kernels."""
    lay = synth.layer(synth.tensor_seed(9, K + N + g), K, N, density=density, layout=layout)
    P = H.pack_layer(lay, g, BN)
    X = _x(lay.seed, M, K)
    Yref, Yabs = H.oracle_result(P, X)
    for streaming_only in (False, True):
        Y = H.run_fused(P, X, streaming_only=streaming_only)
        stats = H.check_tolerances(Y, Yref, Yabs, K)
        assert stats["mean_rel"] < H.MEAN_TOL


@pytest.mark.parametrize("M", [17, 32, 33, 64, 100, 128])
def test_fused_larger_batches(M):
    K, N, g = 1024, 1024, 128
    lay = synth.layer(synth.tensor_seed(9, M), K, N, density=0.01, layout="mixed")
    P = H.pack_layer(lay, g)
    X = _x(lay.seed, M, K)
    Y = H.run_fused(P, X)
    Yref, Yabs = H.oracle_result(P, X)
    H.check_tolerances(Y, Yref, Yabs, K)


# ------------------------------------------------------------------ bit-exact special cases

@pytest.mark.parametrize("BN,g,M", [(256, 128, 8), (128, 64, 16), (256, 64, 32), (256, 128, 1)])
def test_identity_rows_return_the_reconstructed_weights_bit_exact(BN, g, M):
    # X = M rows of the identity: every other addend is exactly 0, so Y row = bf16(W^[k,:] + W_O[k,:])
    K, N = 512, 768
    lay = synth.layer(synth.tensor_seed(8, BN + g), K, N, density=0.03, layout="mixed")
    P = H.pack_layer(lay, g, BN)
    rows = (np.arange(M) * 37 + 5) % K
    hot = np.argsort(lay.mask.sum(axis=1))[::-1][:M // 2]          # include outlier-heavy rows
    rows[:len(hot)] = hot
    X = np.zeros((M, K), dtype=np.uint16)
    X[np.arange(M), rows] = 0x3F80
    Y = H.run_fused(P, X)
    Yref, _ = H.oracle_result(P, X)
    assert np.array_equal(Y, H.f64_to_bf16_bits(Yref))
    # one-hot times a power of two stays exact as well
    X[np.arange(M), rows] = 0x4080                                   # 4.0
    Y = H.run_fused(P, X)
    assert np.array_equal(Y, H.f64_to_bf16_bits(4.0 * Yref))


def test_zero_density_equals_the_dense_kernel_bit_for_bit():
    K, N, g, M = 1024, 1536, 128, 8
    lay = synth.layer(synth.tensor_seed(8, 1), K, N, density=0.0)
    P = H.pack_layer(lay, g)
    X = _x(3, M, K)
    assert np.array_equal(H.run_fused(P, X), H.run_unfused(P, X, with_spmm=False))


@pytest.mark.parametrize("M", [1, 8, 16, 40])
def test_unfused_pair_matches_oracle_and_fused(M):
    K, N, g = 1024, 1024, 128
    lay = synth.layer(synth.tensor_seed(8, 2), K, N, density=0.02, layout="mixed")
    P = H.pack_layer(lay, g)
    X = _x(4, M, K)
    Yd = H.run_unfused(P, X, with_spmm=False)
    Yref_d, Yabs_d = H.oracle_result(P, X, dense_only=True)
    H.check_tolerances(Yd, Yref_d, Yabs_d, K)
    Yu = H.run_unfused(P, X, with_spmm=True)
    Yref, Yabs = H.oracle_result(P, X)
    # the two-kernel path rounds to BF16 twice (the dense result, then the sum): each element may be
    # off by half a BF16 ulp of the dense part plus half an ulp of the total, plus FP32 accumulation
    err = np.abs(H.bits_to_f64(Yu) - Yref)
    bound = 2.0 ** -8 * (np.abs(Yref_d) + np.abs(Yref)) + K * 2.0 ** -24 * Yabs
    assert np.all(err <= bound)
    assert err.sum() / np.abs(Yref).sum() <= 4e-3
    Yf = H.run_fused(P, X)
    H.check_tolerances(Yf, Yref, Yabs, K)


# ------------------------------------------------------------------ edge cases

def test_oversized_tiles_fall_back_to_global_packets():
    # one tile is completely dense in outliers (8192 packets, far above the staged capacity), one
    # row and one column are hot; results must still match
    K, N, g, BN = 256, 512, 128, 256
    lay = synth.layer(synth.tensor_seed(8, 3), K, N, density=0.0)
    mask = np.zeros((K, N), dtype=np.uint8)
    mask[128:256, 0:256] = 1
    mask[3, 256:512] = 1
    mask[0:128, 400] = 1
    kk, nn = np.nonzero(mask)
    rng = np.random.default_rng(0)
    vals = (rng.uniform(0.12, 0.4, size=kk.size) * rng.choice([-1, 1], size=kk.size)).astype(np.float32)
    vb = (vals.view(np.uint32) >> 16).astype(np.uint16)
    lay.mask, lay.coo_k, lay.coo_n, lay.coo_v = mask, kk.astype(np.uint32), nn.astype(np.uint32), vb
    lay.W[kk, nn] = synth.bf16_bits_to_f32(vb)
    P = H.pack_layer(lay, g, BN)
    assert P.L.max_tile_packets == 8192
    for M in (1, 8, 16):
        X = _x(6, M, K)
        Yref, Yabs = H.oracle_result(P, X)
        for streaming_only in (False, True):
            H.check_tolerances(H.run_fused(P, X, streaming_only=streaming_only), Yref, Yabs, K)


def test_several_tails_in_one_strip():
    # Column-slotted packets with tails: in the first 32-column strip of one tile, column 3 has 100
    # outliers, column 12 has 40 and column 27 (same bucket as column 3) has 17; column 5 has exactly
    # 32 (the longest column-slotted list).  A second tile has one long column on top of 1 % noise.
    # Everything fits the staged part, so the tails are read from shared memory.
    K, N, g, BN = 512, 512, 128, 256
    lay = synth.layer(synth.tensor_seed(8, 9), K, N, density=0.01, layout="uniform")
    mask = lay.mask.copy()
    rng = np.random.default_rng(4)
    for col, cnt in ((3, 100), (12, 40), (27, 17), (5, 32)):
        mask[0:128, col] = 0
        mask[rng.choice(128, size=cnt, replace=False), col] = 1
    mask[256 + rng.choice(128, size=77, replace=False), 256 + 130] = 1
    kk, nn = np.nonzero(mask)
    vals = (rng.uniform(0.12, 0.4, size=kk.size) * rng.choice([-1, 1], size=kk.size)).astype(np.float32)
    vb = (vals.view(np.uint32) >> 16).astype(np.uint16)
    lay.mask, lay.coo_k, lay.coo_n, lay.coo_v = mask, kk.astype(np.uint32), nn.astype(np.uint32), vb
    lay.W[kk, nn] = synth.bf16_bits_to_f32(vb)
    P = H.pack_layer(lay, g, BN)
    assert P.L.max_tail_packets == (100 - 4 + 17 - 4 + 3) // 4 and P.L.max_tile_packets < 1024
    for M in (1, 3, 5, 8, 16):
        X = _x(7, M, K)
        Yref, Yabs = H.oracle_result(P, X)
        for streaming_only in (False, True):
            H.check_tolerances(H.run_fused(P, X, streaming_only=streaming_only), Yref, Yabs, K)


@pytest.mark.parametrize("streaming_only", [False, True])
def test_scratch_is_reusable_and_results_are_reproducible(streaming_only):
    K, N, g = 2048, 1024, 128
    lay = synth.layer(synth.tensor_seed(8, 4), K, N, density=0.01, layout="mixed")
    P = H.pack_layer(lay, g)
    outs = []
    for M in (16, 1, 16, 8, 16):
        outs.append((M, H.run_fused(P, _x(5, M, K), streaming_only=streaming_only)))
    a = [y for m, y in outs if m == 16]
    assert np.array_equal(a[0], a[1]) and np.array_equal(a[1], a[2])
    # counters and status word are back to zero (header and every tile-arrival counter)
    head = P.ws[: 256 + 32768].cpu().numpy()
    assert not head.any()


def test_a_reported_device_error_rearms_the_scratch():
    """What a call that gave up leaves behind is put there from the host: an error code in the status word and
    a few arrival counters that never reached their tile's count.  fq_check_status must report the code, clear
    all of it, and the next call on the same scratch must be correct."""
    K, N, g, M = 2048, 1024, 128, 8
    lay = synth.layer(synth.tensor_seed(8, 5), K, N, density=0.01, layout="mixed")
    P = H.pack_layer(lay, g)
    words = P.ws[: 256 + 32768].view(torch.int32)
    words[0] = fq.FQ_ERR_TIMEOUT
    words[64 + 0] = 3            # strip 0 of tile 0
    words[64 + 9] = 1            # strip 1 of tile 1
    words[64 + 8 * 3 + 7] = 2
    with pytest.raises(fq.FqError) as e:
        fq.fq_check_status(P.ws)
    assert e.value.code == fq.FQ_ERR_TIMEOUT
    assert not P.ws[: 256 + 32768].cpu().numpy().any()
    X = _x(5, M, K)
    Yref, Yabs = H.oracle_result(P, X)
    H.check_tolerances(H.run_fused(P, X, streaming_only=True), Yref, Yabs, K)


@pytest.mark.parametrize("M", [4, 16, 24])
def test_a_layout_that_does_not_belong_to_the_arrays_is_reported_not_faulted(M):
    """Bucket descriptors that point past the packets a stage holds (here: max_tile_packets lowered by hand, as
    after re-encoding denser outliers with an old layout struct) must end in FQ_ERR_FORMAT, not in a read
    outside shared memory.  (The streaming kernels stage packets; the short-job kernel reads them from global
    memory and does not depend on that field.)"""
    K, N, g = 1024, 512, 128
    lay = synth.layer(synth.tensor_seed(8, 6), K, N, density=0.03, layout="uniform")
    P = H.pack_layer(lay, g)
    assert P.L.max_tile_packets > 16 and P.L.max_tail_packets == 0
    good = P.L.max_tile_packets
    P.L.max_tile_packets = 8
    P.L.kernel_hint = 1
    try:
        X = H.to_dev(_x(5, M, K))
        Y = torch.zeros((M, N), dtype=torch.int16, device="cuda")
        fq.fq_fused_w4a16_outlier_gemm(P.L, X, M, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"], P.d["info"],
                                       P.d["packed"], Y, P.ws)
        with pytest.raises(fq.FqError) as e:
            fq.fq_check_status(P.ws)
        assert e.value.code == fq.FQ_ERR_FORMAT
    finally:
        P.L.max_tile_packets = good
        P.L.kernel_hint = 0
    Yref, Yabs = H.oracle_result(P, _x(5, M, K))
    H.check_tolerances(H.run_fused(P, _x(5, M, K)), Yref, Yabs, K)
    H.check_tolerances(H.run_fused(P, _x(5, M, K), streaming_only=True), Yref, Yabs, K)


@pytest.mark.parametrize("M", [1, 8, 16])
@pytest.mark.parametrize("streaming_only", [False, True])
def test_a_bucket_descriptor_past_its_tile_is_reported_not_followed(M, streaming_only):
    """A corrupt descriptor (a depth that reaches past the packets of its tile) is skipped and reported by
    every kernel: neither the short-job kernel (packets from global memory) nor the streaming kernels (packets
    staged in shared memory) follow it."""
    K, N, g = 512, 512, 128
    lay = synth.layer(synth.tensor_seed(8, 7), K, N, density=0.01, layout="uniform")
    P = H.pack_layer(lay, g)
    info = P.info.copy()
    info[-1] = (info[-1] & 0xffff) | (255 << 16)            # last bucket of the last tile: 255 packets deep
    bad = H.to_dev(info)
    P.L.kernel_hint = 1 if streaming_only else 0
    try:
        X = H.to_dev(_x(5, M, K))
        Y = torch.zeros((M, N), dtype=torch.int16, device="cuda")
        fq.fq_fused_w4a16_outlier_gemm(P.L, X, M, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"], bad,
                                       P.d["packed"], Y, P.ws)
        with pytest.raises(fq.FqError) as e:
            fq.fq_check_status(P.ws)
        assert e.value.code == fq.FQ_ERR_FORMAT
    finally:
        P.L.kernel_hint = 0
    Yref, Yabs = H.oracle_result(P, _x(5, M, K))
    H.check_tolerances(H.run_fused(P, _x(5, M, K), streaming_only=streaming_only), Yref, Yabs, K)


@pytest.mark.parametrize("M", [1, 8, 16, 24])
def test_many_units_per_cta_are_repeatable(M):
    # several units per CTA with split tiles: at M = 24 the sparse warps of the large-batch kernel
    # work on different row tiles of one column tile at the same time
    K, N, g = 4096, 6144, 128
    lay = synth.layer(synth.tensor_seed(8, 6), K, N, density=0.01, layout="mixed")
    P = H.pack_layer(lay, g)
    X = _x(9, M, K)
    Y = H.run_fused(P, X)
    for _ in range(3):
        assert np.array_equal(H.run_fused(P, X), Y)
    cols = np.arange(0, N, 24, dtype=np.uint32)
    Yref, Yabs = H.oracle_result(P, X, cols=cols)
    H.check_tolerances(Y[:, cols], Yref, Yabs, K)


def _with_fp16_values(lay, seed):
    """The layer's outlier positions with values re-drawn as IEEE binary16 numbers (ten fraction bits in use)."""
    rng = np.random.default_rng(seed)
    vals = (rng.uniform(0.12, 0.4, size=lay.coo_k.size) * rng.choice([-1, 1], size=lay.coo_k.size)).astype(np.float16)
    lay.coo_v = vals.view(np.uint16).copy()
    lay.W[lay.coo_k, lay.coo_n] = vals.astype(np.float32)
    return lay


@pytest.mark.parametrize("M", [1, 4, 8, 16, 24])
def test_fp16_outlier_values_match_the_oracle(M):
    """Outlier values of the second type of Table 1 (IEEE binary16), every element, through every kernel that
    serves the shape (M = 24: the tcgen05 kernel)."""
    K, N, g = 1024, 768, 128
    lay = _with_fp16_values(synth.layer(synth.tensor_seed(8, 11), K, N, density=0.02, layout="mixed"), 21)
    P = H.pack_layer(lay, g, value_type=fq.FQ_VALUE_FP16)
    X = _x(12, M, K)
    Yref, Yabs = H.oracle_result(P, X)
    for streaming_only in (False, True):
        H.check_tolerances(H.run_fused(P, X, streaming_only=streaming_only), Yref, Yabs, K)
    # the unfused pair reads the same slots; it rounds to BF16 twice (the dense result, then the sum)
    Yref_d, _ = H.oracle_result(P, X, dense_only=True)
    err = np.abs(H.bits_to_f64(H.run_unfused(P, X)) - Yref)
    assert np.all(err <= 2.0 ** -8 * (np.abs(Yref_d) + np.abs(Yref)) + K * 2.0 ** -24 * Yabs)


@pytest.mark.parametrize("M", [1, 8, 16, 24])
def test_fp16_outlier_values_keep_their_ten_fraction_bits(M):
    """Two outliers in one column, 1 + 2^-9 and -1, activations 512 in both rows, nothing else: Y is exactly 1.
    With the first value cut to BF16 (eight significant bits) it would be 0."""
    K, N, g = 256, 512, 128
    lay = synth.layer(1, K, N, density=0.0)
    lay.W[:] = 0.0
    cols = np.array([5, 5, 300, 300], dtype=np.uint32)
    rows = np.array([3, 200, 77, 130], dtype=np.uint32)
    vals = np.array([1 + 2.0 ** -9, -1.0, -(1 + 2.0 ** -10), 1.0], dtype=np.float16)
    mask = np.zeros((K, N), dtype=np.uint8)
    mask[rows, cols] = 1
    lay.mask, lay.coo_k, lay.coo_n, lay.coo_v = mask, rows, cols, vals.view(np.uint16).copy()
    lay.W[rows, cols] = vals.astype(np.float32)
    P = H.pack_layer(lay, g, value_type=fq.FQ_VALUE_FP16)
    Xf = np.zeros((M, K), dtype=np.float32)
    Xf[:, rows] = 512.0
    X = (Xf.view(np.uint32) >> 16).astype(np.uint16)
    for streaming_only in (False, True):
        Y = H.bits_to_f64(H.run_fused(P, X, streaming_only=streaming_only))
        assert np.all(Y[:, 5] == 1.0) and np.all(Y[:, 300] == -0.5)
        Y[:, [5, 300]] = 0
        assert not Y.any()


@pytest.mark.parametrize("M", [1, 8, 16, 24])
def test_layer_with_repurposed_pad_slots_matches_the_oracle(M):
    """Section 3.2.1's remark: every padding slot of the column-slotted packets holds an original weight.  Same
    packet count, every slot live; every element against the oracle through each kernel."""
    K, N, g = 1024, 768, 128
    lay = synth.layer(synth.tensor_seed(8, 12), K, N, density=0.01, layout="mixed")
    L0 = fq.fq_get_layout(K, N, g)
    before = fq.fq_encode_tilecoo(L0, lay.coo_k, lay.coo_n, lay.coo_v)[2].shape[0]
    mask2, added = fq.fq_repurpose_pad_slots(L0, lay.W, lay.mask)
    assert added > 0
    kk, nn = np.nonzero(mask2)
    lay.mask, lay.coo_k, lay.coo_n = mask2, kk.astype(np.uint32), nn.astype(np.uint32)
    lay.coo_v = H.f64_to_bf16_bits(lay.W[kk, nn].astype(np.float64))
    P = H.pack_layer(lay, g)
    assert P.packed.shape[0] == before
    X = _x(13, M, K)
    Yref, Yabs = H.oracle_result(P, X)
    for streaming_only in (False, True):
        H.check_tolerances(H.run_fused(P, X, streaming_only=streaming_only), Yref, Yabs, K)


def test_column_shards_computed_one_after_the_other_give_the_full_result():
    """The N-sharded wrapper's per-rank part on one GPU: the two ranks' shards of a layer (widths 512 and 256) are
    packed and run one after the other, without a collective, and their slices side by side are the full Y."""
    from paper_2608_15531_b200.sharded import ShardedLayer
    K, N, g, M = 512, 768, 128, 8
    lay = synth.layer(synth.tensor_seed(8, 13), K, N, density=0.01, layout="mixed")
    X = _x(14, M, K)
    P = H.pack_layer(lay, g)
    Yref, Yabs = H.oracle_result(P, X)
    Xd = H.to_dev(X)
    parts = []
    for rank in range(2):
        layer = ShardedLayer(lay.W, lay.mask, lay.coo_k, lay.coo_n, lay.coo_v, g, rank, 2)
        parts.append(H.bf16_bits(layer.local(Xd)))
    Y = np.concatenate(parts, axis=1)
    assert np.array_equal(Y, H.run_fused(P, X))          # same kernels, same per-column arithmetic: bit-equal
    H.check_tolerances(Y, Yref, Yabs, K)
    one = ShardedLayer(lay.W, lay.mask, lay.coo_k, lay.coo_n, lay.coo_v, g, 0, 1)
    assert np.array_equal(H.bf16_bits(one.forward(Xd)), Y)


@pytest.mark.parametrize("K,N,g", [(128, 128, 128), (128, 256, 64), (256, 128, 128), (8192, 256, 128)])
@pytest.mark.parametrize("M", [1, 4, 7, 16])
def test_smallest_and_thinnest_layers(K, N, g, M):
    """One k-step (most warps of a short-job CTA have nothing to do), one column tile, one strip per CTA with 64
    k-steps: the extremes of the short-job kernel's split, and the same shapes through the streaming kernel."""
    lay = synth.layer(synth.tensor_seed(8, K + N), K, N, density=0.02, layout="uniform")
    P = H.pack_layer(lay, g)
    X = _x(15, M, K)
    Yref, Yabs = H.oracle_result(P, X)
    for streaming_only in (False, True):
        H.check_tolerances(H.run_fused(P, X, streaming_only=streaming_only), Yref, Yabs, K)


def test_argument_errors_launch_nothing():
    K, N, g = 512, 512, 128
    lay = synth.layer(1, K, N, density=0.01)
    P = H.pack_layer(lay, g)
    X = H.to_dev(_x(1, 4, K))
    Y = torch.zeros((4, N), dtype=torch.int16, device="cuda")
    with pytest.raises(fq.FqError) as e:
        fq.fq_fused_w4a16_outlier_gemm(P.L, X, 0, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"], P.d["info"],
                                       P.d["packed"], Y, P.ws)
    assert e.value.code == fq.FQ_ERR_INVALID_ARG
    small = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(fq.FqError) as e:
        fq.fq_fused_w4a16_outlier_gemm(P.L, X, 4, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"], P.d["info"],
                                       P.d["packed"], Y, small)
    assert e.value.code == fq.FQ_ERR_BUFFER_TOO_SMALL
    with pytest.raises(fq.FqError) as e:
        fq.fq_fused_w4a16_outlier_gemm(P.L, None, 4, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"],
                                       P.d["info"], P.d["packed"], Y, P.ws)
    assert e.value.code == fq.FQ_ERR_INVALID_ARG
    assert not Y.any()


def test_host_io_entry_point_matches_device_entry_point():
    K, N, g, M = 1024, 1024, 128, 16
    lay = synth.layer(synth.tensor_seed(8, 5), K, N, density=0.01, layout="mixed")
    P = H.pack_layer(lay, g)
    Xb = _x(7, M, K)
    Y_dev = H.run_fused(P, Xb)
    xh = torch.from_numpy(Xb.view(np.int16)).pin_memory()
    yh = torch.zeros((M, N), dtype=torch.int16).pin_memory()
    xd = torch.empty((M, K), dtype=torch.int16, device="cuda")
    yd = torch.empty((M, N), dtype=torch.int16, device="cuda")
    fq.fq_fused_host_io(P.L, xh, M, xd, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"], P.d["info"],
                        P.d["packed"], yd, yh, P.ws)
    assert np.array_equal(yh.numpy().view(np.uint16), Y_dev)
    # the asynchronous form: two calls enqueued, one synchronisation
    yh2 = torch.zeros((M, N), dtype=torch.int16).pin_memory()
    yd2 = torch.empty((M, N), dtype=torch.int16, device="cuda")
    xd2 = torch.empty((M, K), dtype=torch.int16, device="cuda")
    yh.zero_()
    for (a_x, a_y, a_yh) in ((xd, yd, yh), (xd2, yd2, yh2)):
        fq.fq_fused_host_io_async(P.L, xh, M, a_x, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"], P.d["info"],
                                  P.d["packed"], a_y, a_yh, P.ws)
    torch.cuda.synchronize()
    assert np.array_equal(yh.numpy().view(np.uint16), Y_dev) and np.array_equal(yh2.numpy().view(np.uint16), Y_dev)


# ------------------------------------------------------------------ full-size layers, every output column

FULL = [("8b_" + n, 2, i, K, N) for i, (n, K, N) in enumerate(synth.LLAMA3_8B)]


@pytest.mark.parametrize("name,cfg,idx,K,N", FULL)
def test_full_size_layers_every_column(name, cfg, idx, K, N):
    """The benchmark's own layers in the launch configuration the benchmark times (M = 1, 8, 16), every
    element of Y against the oracle."""
    g = 128
    lay = synth.layer(synth.tensor_seed(cfg, idx), K, N, density=0.01, layout="mixed")
    P = H.pack_layer(lay, g)
    for M in (1, 8, 16):
        X = _x(lay.seed, M, K)
        Y = H.run_fused(P, X)
        Yref, Yabs = H.oracle_result(P, X)
        res = H.check_tolerances(Y, Yref, Yabs, K)
        if M >= 8:
            assert res["fallback_cols"] == 0, res


def _sample_cols(lay, N, seed, n_random=64):
    """First and last columns, random ones, and the columns richest in outliers."""
    rng = np.random.default_rng(seed)
    return np.unique(np.concatenate([np.arange(0, 8), np.arange(N - 8, N), rng.integers(0, N, n_random),
                                     np.argsort(lay.mask.sum(axis=0))[::-1][:8]])).astype(np.uint32)


# ------------------------------------------------------------------ outlier-density sweep (configuration 3)

@pytest.mark.parametrize("layout", ["uniform", "clustered"])
@pytest.mark.parametrize("density", [0.0, 0.005, 0.01, 0.02, 0.05])
def test_density_sweep_on_sampled_columns(density, layout):
    K, N, g, M = 4096, 14336, 128, 8
    if density == 0.0 and layout == "clustered":
        pytest.skip("no outliers: one layout is enough")
    lay = synth.layer(synth.tensor_seed(3, int(density * 1000) + (layout == "clustered")), K, N, density=density,
                      layout=layout)
    P = H.pack_layer(lay, g)
    cols = _sample_cols(lay, N, 3)
    X = _x(lay.seed, M, K)
    Y = H.run_fused(P, X)
    Yref, Yabs = H.oracle_result(P, X, cols=cols)
    H.check_tolerances(Y[:, cols], Yref, Yabs, K)
    # the unfused pair computes the same thing (one more BF16 rounding of the dense half)
    Yu = H.run_unfused(P, X)
    Yd, _ = H.oracle_result(P, X, cols=cols, dense_only=True)
    bound = 2.0 ** -8 * (np.abs(Yd) + np.abs(Yref)) + K * 2.0 ** -24 * Yabs
    assert np.all(np.abs(H.bits_to_f64(Yu[:, cols]) - Yref) <= bound)


# ------------------------------------------------------------------ LLaMA-3-70B shapes (configuration 4)

@pytest.mark.parametrize("idx", range(len(synth.LLAMA3_70B)))
def test_llama3_70b_layers_on_sampled_columns(idx):
    name, K, N = synth.LLAMA3_70B[idx]
    g = 128
    lay = synth.layer(synth.tensor_seed(4, idx), K, N, density=0.01, layout="mixed")
    P = H.pack_layer(lay, g)
    cols = _sample_cols(lay, N, idx, n_random=48)
    for M in (1, 4, 16, 32):
        X = _x(lay.seed, M, K)
        Y = H.run_fused(P, X)
        Yref, Yabs = H.oracle_result(P, X, cols=cols)
        H.check_tolerances(Y[:, cols], Yref, Yabs, K)


# ------------------------------------------------------------------ batch transition sweep (configuration 5)

@pytest.mark.parametrize("g", [64, 128])
def test_batch_transition_sweep_on_sampled_columns(g):
    K, N = 8192, 28672
    lay = synth.layer(synth.tensor_seed(5, g), K, N, density=0.01, layout="mixed")
    P = H.pack_layer(lay, g)
    cols = _sample_cols(lay, N, g, n_random=40)
    for M in (1, 2, 4, 8, 16, 32, 64, 128):
        X = _x(lay.seed, M, K)
        Y = H.run_fused(P, X)
        Yref, Yabs = H.oracle_result(P, X, cols=cols)
        H.check_tolerances(Y[:, cols], Yref, Yabs, K)


# ------------------------------------------------------------------ tile counts of the paper's largest operator

@pytest.mark.parametrize("K,N", [(14848, 2304), (75264, 512)])
def test_tile_counts_that_are_not_powers_of_two_on_sampled_columns(K, N):
    # 14848 = 116 row tiles and 75264 = 588 row tiles (the two orientations of the largest operator in the
    # paper's Table of shapes), with few column tiles so that the host side stays small: unit ranges that
    # start and end anywhere inside a tile, and tiles shared by many CTAs
    g = 128
    lay = synth.layer(synth.tensor_seed(6, K % 97), K, N, density=0.02, layout="uniform")
    P = H.pack_layer(lay, g)
    cols = _sample_cols(lay, N, 6, n_random=40)
    for M in (1, 8, 16, 32):
        X = _x(lay.seed, M, K)
        Y = H.run_fused(P, X)
        Yref, Yabs = H.oracle_result(P, X, cols=cols)
        H.check_tolerances(Y[:, cols], Yref, Yabs, K)


# ------------------------------------------------------------------ ordering of dependent calls

@pytest.mark.parametrize("M", [1, 8, 16])
def test_back_to_back_dependent_calls_keep_stream_order(M):
    """The small-batch kernel may start while the kernel before it in the stream is draining.  A call
    whose activations are the previous call's output must still see all of it: chain three calls
    Y1 = f(X), Y2 = f(Y1), Y3 = f(Y2) without any synchronisation in between and compare every link
    with the oracle applied to the link's actual input."""
    K = N = 2048
    g = 128
    lay = synth.layer(synth.tensor_seed(8, 77), K, N, density=0.01, layout="mixed")
    P = H.pack_layer(lay, g)
    X0 = H.to_dev(_x(5, M, K))
    Ys = [torch.full((M, N), 0x7fc0, dtype=torch.int16, device="cuda") for _ in range(3)]
    for rep in range(5):
        src = X0
        for Y in Ys:
            fq.fq_fused_w4a16_outlier_gemm(P.L, src, M, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"],
                                           P.d["info"], P.d["packed"], Y, P.ws)
            src = Y
        fq.fq_check_status(P.ws)
        chain = [X0] + Ys
        for a, b in zip(chain[:-1], chain[1:]):
            xin = a.cpu().numpy().view(np.uint16)
            Yref, Yabs = H.oracle_result(P, xin)
            H.check_tolerances(b.cpu().numpy().view(np.uint16), Yref, Yabs, K)
        for Y in Ys:
            Y.fill_(0x7fc0)
