"""The seeded generator: determinism, counts and the three outlier layouts.  CPU only."""
import numpy as np

from paper_2608_15531_b200 import synth


def test_layer_is_deterministic_and_counts_match():
    a = synth.layer(synth.tensor_seed(1, 0), 256, 512, density=0.01, layout="mixed")
    b = synth.layer(synth.tensor_seed(1, 0), 256, 512, density=0.01, layout="mixed")
    assert np.array_equal(a.W, b.W) and np.array_equal(a.mask, b.mask)
    assert a.nnz == round(0.01 * 256 * 512) == int(a.mask.sum())
    assert np.array_equal(a.mask[a.coo_k, a.coo_n], np.ones(a.nnz, dtype=np.uint8))
    # the dense matrix carries the BF16 outlier values
    assert np.array_equal(a.W[a.coo_k, a.coo_n], synth.bf16_bits_to_f32(a.coo_v))
    mag = np.abs(synth.bf16_bits_to_f32(a.coo_v))
    assert mag.min() >= 6 * 0.02 * 0.99 and mag.max() <= 20 * 0.02 * 1.01
    c = synth.layer(synth.tensor_seed(1, 1), 256, 512, density=0.01, layout="mixed")
    assert not np.array_equal(a.W, c.W)


def test_dense_weights_and_activations_have_the_stated_moments():
    L = synth.layer(5, 512, 512, density=0.0)
    assert L.nnz == 0
    assert abs(float(L.W.std()) - 0.02) < 2e-4 and abs(float(L.W.mean())) < 2e-4
    X = synth.bf16_bits_to_f32(synth.activations(5, 16, 4096))
    assert abs(float(X.std()) - 1.0) < 0.02
    X8 = synth.activations(5, 8, 4096)
    assert np.array_equal(X8, synth.activations(5, 16, 4096)[:8])


def test_mixed_layout_concentrates_half_in_hot_rows():
    L = synth.layer(9, 1024, 512, density=0.01, layout="mixed")
    per_row = L.mask.sum(axis=1)
    hot = np.sort(per_row)[::-1][:11]              # ceil(0.01 * 1024) = 11 hot rows
    assert hot.sum() >= 0.45 * L.nnz
    assert abs(L.hot_fraction - 0.5) < 0.01


def test_clustered_layout_caps_the_hot_region():
    K, N = 1024, 2048
    for rho in (0.005, 0.05):
        L = synth.layer(11, K, N, density=rho, layout="clustered")
        assert L.nnz == round(rho * K * N)
        cap = 5 * N + 10 * K - 50
        assert L.hot_fraction <= 0.8 + 1.0 / L.nnz
        assert L.hot_fraction * L.nnz <= 0.75 * cap + 1
    assert L.hot_fraction < 0.8                    # 5 %: the cap binds


def test_uniform_layout_is_flat():
    L = synth.layer(13, 512, 512, density=0.02, layout="uniform")
    per_row = L.mask.sum(axis=1)
    assert per_row.max() < 4 * per_row.mean()
