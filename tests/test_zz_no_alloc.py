"""The entry point for callers that may not allocate device memory: same result as the entry point
that takes a caller-allocated workspace, call after call.  Collected last on purpose (file name),
so a run that stops at the first failure has already exercised everything else.  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_2608_15531_b200 import binding as fq
from paper_2608_15531_b200 import synth

import harness as H

pytestmark = pytest.mark.gpu


def _run_noalloc(P, X_bits):
    M = X_bits.shape[0]
    X = H.to_dev(X_bits)
    Y = torch.full((M, P.L.N), 0x7fc0, dtype=torch.int16, device="cuda")   # NaN pattern: all of Y must be written
    fq.fq_fused_w4a16_outlier_gemm_noalloc(P.L, X, M, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"],
                                           P.d["info"], P.d["packed"], Y)
    torch.cuda.synchronize()
    return H.bf16_bits(Y)


def test_noalloc_entry_point_matches_the_workspace_entry_point_twice_in_a_row():
    # a layer whose tiles are shared between CTAs, so the scratch (partials, arrival counters) is used
    K, N, g = 2048, 1536, 128
    lay = synth.layer(synth.tensor_seed(7, 1), K, N, density=0.01, layout="mixed")
    P = H.pack_layer(lay, g)
    for M in (16, 5):
        X = synth.activations(lay.seed + M, M, K)
        want = H.run_fused(P, X)                     # existing entry point, caller-allocated scratch
        first = _run_noalloc(P, X)
        second = _run_noalloc(P, X)                  # finds the first call's leftovers in the shared array
        # same kernel, same fixed summation order: the tolerance of the parity tests is met with zero error
        assert np.array_equal(first, want)
        assert np.array_equal(second, want)
        Yref, Yabs = H.oracle_result(P, X)
        H.check_tolerances(second, Yref, Yabs, K)


def test_noalloc_entry_point_refuses_what_does_not_fit():
    K, N, g = 512, 512, 128
    lay = synth.layer(3, K, N, density=0.01)
    P = H.pack_layer(lay, g)
    M = 17                                           # needs twice the scratch of M <= 16
    X = H.to_dev(synth.activations(1, M, K))
    Y = torch.zeros((M, N), dtype=torch.int16, device="cuda")
    with pytest.raises(fq.FqError) as e:
        fq.fq_fused_w4a16_outlier_gemm_noalloc(P.L, X, M, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"],
                                               P.d["info"], P.d["packed"], Y)
    assert e.value.code == fq.FQ_ERR_BUFFER_TOO_SMALL
    assert "scratch" in str(e.value)
    torch.cuda.synchronize()
    assert not Y.any()


def test_noalloc_entry_point_reports_argument_errors_before_it_touches_the_stream():
    K, N, g, M = 512, 512, 128, 4
    lay = synth.layer(3, K, N, density=0.01)
    P = H.pack_layer(lay, g)
    Y = torch.full((M, N), 0x1234, dtype=torch.int16, device="cuda")
    with pytest.raises(fq.FqError) as e:
        fq.fq_fused_w4a16_outlier_gemm_noalloc(P.L, None, M, P.d["wq"], P.d["scale"], P.d["zero"], P.d["indptr"],
                                               P.d["info"], P.d["packed"], Y)
    assert e.value.code == fq.FQ_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert bool((Y == 0x1234).all())
