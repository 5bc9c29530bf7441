"""GPU parity for the error-measurement kernels: fp64 reference product and the reductions."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_26077_b200 import fmm, workloads as Wl
from gpu_common import dev

pytestmark = pytest.mark.gpu


def test_ref_gemm_fp64_matches_oracle():
    A, B = Wl.gaussian(192, 272, 320, 2)
    got = fmm.fmm_ref_gemm_fp64(dev(A), dev(B)).cpu().numpy()
    want = O.ref_gemm(A, B)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-12)


def test_error_stats_match_oracle():
    rng = np.random.default_rng(0)
    Cm = rng.standard_normal((384, 250)).astype(np.float32)
    Cr = Cm.astype(np.float64) + 1e-2 * rng.standard_normal((384, 250))
    Cr[17, 33] += 5.0
    got = fmm.fmm_error_stats(dev(Cm), dev(Cr)).cpu().numpy()
    want = O.error_stats(Cm.astype(np.float64), Cr)
    assert got[0] == pytest.approx(want[0], rel=1e-12)
    assert got[1] == pytest.approx(want[1], rel=1e-12)
    assert got[2] == want[2]
    again = fmm.fmm_error_stats(dev(Cm), dev(Cr)).cpu().numpy()
    assert np.array_equal(got, again)          # deterministic reduction
