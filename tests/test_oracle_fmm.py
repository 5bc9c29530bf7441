"""Pins for the oracle's fused fast matmul: exactness without quantization, the cubic special
case, the paper's printed error figures, the Phi-predicted ratios, the Rademacher reversal."""
import math

import numpy as np
import pytest

from oracle import oracle as O
from oracle import realizations as R
from paper_2609_26077_b200 import workloads as Wl


def coeffs(name):
    return [np.array(R.to_float(x), dtype=np.float32) for x in R.NAMED[name]()]


def brute_force(A, B):
    M, K = A.shape
    N = B.shape[1]
    C = [[0.0] * N for _ in range(M)]
    for i in range(M):
        for j in range(N):
            s = 0.0
            for k in range(K):
                s += float(A[i, k]) * float(B[k, j])
            C[i][j] = s
    return np.array(C)


def test_reference_gemm_is_the_plain_definition():
    A, B = Wl.gaussian(6, 5, 7, 0)
    assert np.allclose(O.ref_gemm(A, B), brute_force(A, B), rtol=1e-14, atol=1e-14)
    A, B = Wl.gaussian(96, 160, 64, 1)
    lib = A.astype(np.float64) @ B.astype(np.float64)
    assert np.allclose(O.ref_gemm(A, B), lib, rtol=1e-13, atol=1e-13)
    rows = [0, 17, 95]
    assert np.array_equal(O.ref_gemm_rows(A, B, rows), O.ref_gemm(A, B)[rows])


@pytest.mark.parametrize("name", ["strassen", "winograd", "cubic"])
@pytest.mark.parametrize("levels", [1, 2, 3])
def test_unquantized_algorithm_equals_product_exactly(name, levels):
    # integer-valued inputs make every fp32 combination exact, so the bilinear algorithm must
    # reproduce A*B exactly; rectangular shapes catch transposed operands or quadrants
    U, V, W = coeffs(name)
    d = 1 << levels
    M, K, N = 3 * d, 2 * d, 5 * d
    A, B = Wl.small_integers(M, K, N, seed=levels)
    C = O.fused_fmm(A, B, U, V, W, levels=levels, mode=O.SCALE_IDENTITY)
    assert np.array_equal(C, brute_force(A, B))


def test_unquantized_optimum_equals_product_to_rounding():
    U, V, W = coeffs("phi_optimal")
    for levels in (1, 2):
        A, B = Wl.gaussian(8 * levels, 12 * levels, 4 * levels, 3)
        C = O.fused_fmm(A, B, U, V, W, levels=levels, mode=O.SCALE_IDENTITY)
        ref = O.ref_gemm(A, B)
        assert np.linalg.norm(C - ref) / np.linalg.norm(ref) < 2e-6   # fp32 coefficients and combos


@pytest.mark.parametrize("mode", [O.SCALE_FP32, O.SCALE_UE8M0])
def test_cubic_fp8_is_product_of_dequantized_operands(mode):
    A, B = Wl.gaussian(64, 128, 96, 4)
    ca, sa, _ = O.quant_rows(A, 32, mode)
    cb, sb, _ = O.quant_cols(B, 32, mode)
    want = O.dequant_rows(ca, sa, 32) @ O.dequant_cols(cb, sb, 32)
    got = O.fused_fmm(A, B, levels=0, blk=32, mode=mode)
    assert np.allclose(got, want, rtol=1e-13, atol=1e-13)


def test_rank8_realization_reproduces_cubic_fp8():
    # blocks never straddle a quadrant boundary, so the rank-8 realization at one level quantizes
    # exactly the same blocks as the cubic product; only the fp64 summation order differs
    U, V, W = coeffs("cubic")
    A, B = Wl.gaussian(128, 256, 64, 5)
    c8 = O.fused_fmm(A, B, U, V, W, levels=1, blk=32)
    c0 = O.fused_fmm(A, B, levels=0, blk=32)
    assert np.allclose(c8, c0, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("levels", [1, 2])
def test_fused_result_is_decoded_sum_of_leaf_products(levels):
    # the quantized leaf operands returned for bit parity are the ones the product is made of
    U, V, W = coeffs("winograd")
    n = 64 * (1 << levels)
    A, B = Wl.gaussian(n, n, n, 6)
    ca, sa, _ = O.encode(A, "A", U, V, levels)
    cb, sb, _ = O.encode(B, "B", U, V, levels)
    T = 7 ** levels
    assert ca.shape[0] == T and cb.shape[0] == T
    leaf = [O.dequant_rows(ca[t], sa[t], 32) @ O.dequant_cols(cb[t], sb[t], 32) for t in range(T)]

    def decode(terms, lv):
        if lv == 0:
            return terms[0]
        per = len(terms) // 7
        Ms = [decode(terms[r * per:(r + 1) * per], lv - 1) for r in range(7)]
        h = Ms[0].shape[0]
        C = np.zeros((2 * h, 2 * Ms[0].shape[1]))
        w = Ms[0].shape[1]
        for q in range(4):
            blk = sum(float(W[r][q]) * Ms[r] for r in range(7))
            C[(q >> 1) * h:(q >> 1) * h + h, (q & 1) * w:(q & 1) * w + w] = blk
        return C

    want = decode(leaf, levels)
    got = O.fused_fmm(A, B, U, V, W, levels=levels, blk=32)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("mode,blk", [(O.SCALE_FP32, 32), (O.SCALE_UE8M0, 32), (O.SCALE_FP32, 128)])
def test_sampled_leaf_product_equals_entries_of_the_whole_product(mode, blk):
    # the sampled-entry routine used at full size: its entries are those of the cubic fp8 product (one leaf),
    # bit for bit (same dequantization, same summation order), and a brute-force sum in Python agrees
    A, B = Wl.gaussian(96, 128, 256, 7)
    ca, sa, _ = O.quant_rows(A, blk, mode)
    cb, sb, _ = O.quant_cols(B, blk, mode)
    rows, cols = [0, 5, 17, 95], [3, 64, 65, 127, 8]
    got = O.leaf_product_sample(ca, sa, cb, sb, blk, rows, cols)
    whole = O.fused_fmm(A, B, levels=0, blk=blk, mode=mode)
    assert np.array_equal(got, whole[np.ix_(rows, cols)])
    da, db = O.dequant_rows(ca, sa, blk), O.dequant_cols(cb, sb, blk)
    brute = brute_force(da[rows], db[:, cols])
    assert np.allclose(got, brute, rtol=1e-14, atol=1e-14)
    # a transposed or shifted index would be caught: entries of different rows / columns differ
    assert not np.allclose(got[0], got[1]) and not np.allclose(got[:, 0], got[:, 1])


def _mean_errors(family, n, blk, levels, seeds, names=("cubic", "strassen", "winograd", "phi_optimal"),
                 mode=O.SCALE_FP32):
    out = {k: [] for k in names}
    for seed in seeds:
        A, B = family(n, n, n, seed)
        ref = O.ref_gemm(A, B)
        for name in names:
            U, V, W = coeffs(name)
            lv = 0 if name == "cubic" else levels
            out[name].append(O.rel_frobenius(O.fused_fmm(A, B, U, V, W, levels=lv, blk=blk, mode=mode), ref))
    return {k: float(np.mean(v)) for k, v in out.items()}


def test_paper_emulated_error_figures_blk128_signed_uniform():
    # Table E.1 row <2,2,2>: blk128, signed-uniform operands, block edge 256 (n = 512), one level,
    # eight paired samples: e_lib/e_cub = 2.4486 at e_lib = 0.0874 gives e_cubic = 0.03569;
    # re-based (Phi-optimal) / cubic = 1.7190.  App. D: s_q ~ 0.0253 predicts e_cubic ~ s_q sqrt 2.
    from golden_values import figures
    g = figures()                    # tests/golden/printed_figures.json
    e = _mean_errors(Wl.uniform, 512, 128, 1, range(8))
    assert e["cubic"] == pytest.approx(g["e_lib_222"] / g["e_lib_over_e_cubic_222"], rel=0.02)
    assert e["cubic"] == pytest.approx(g["s_q"] * math.sqrt(2), rel=0.02)
    assert e["phi_optimal"] / e["cubic"] == pytest.approx(g["rebased_over_cubic_222"], rel=0.02)
    # Phi-predicted ordering and magnitudes (Sec. 3): 5/3 < 2 < sqrt 7
    assert e["strassen"] / e["cubic"] == pytest.approx(2.0, rel=0.04)
    assert e["winograd"] / e["cubic"] == pytest.approx(math.sqrt(7), rel=0.04)
    assert e["cubic"] < e["phi_optimal"] < e["strassen"] < e["winograd"]


def test_ratios_follow_sqrt_phi_over_8_blk32_gaussian():
    e = _mean_errors(Wl.gaussian, 256, 32, 1, range(6))
    assert e["phi_optimal"] / e["cubic"] == pytest.approx(5 / 3, rel=0.03)
    assert e["strassen"] / e["cubic"] == pytest.approx(2.0, rel=0.03)
    assert e["winograd"] / e["cubic"] == pytest.approx(math.sqrt(7), rel=0.03)


def test_recursion_ratio_is_power_of_one_level_ratio():
    # Sec. 3: predicted RMS ratio (5/3)^l under recursion; Strassen 2^l
    e = _mean_errors(Wl.gaussian, 256, 32, 2, range(3), names=("cubic", "strassen", "phi_optimal"))
    assert e["phi_optimal"] / e["cubic"] == pytest.approx((5 / 3) ** 2, rel=0.05)
    assert e["strassen"] / e["cubic"] == pytest.approx(4.0, rel=0.05)


def test_ue8m0_mode_keeps_ratios():
    e = _mean_errors(Wl.gaussian, 256, 32, 1, range(4), mode=O.SCALE_UE8M0)
    assert e["phi_optimal"] / e["cubic"] == pytest.approx(5 / 3, rel=0.04)
    assert e["strassen"] / e["cubic"] == pytest.approx(2.0, rel=0.04)


def test_rademacher_operands_reverse_the_order():
    # Sec. 4.3 / Table E.8: on +-1 operands classic Strassen beats the Phi-optimal realization
    # (its combinations are small integers, exactly representable after block scaling)
    A, B = Wl.rademacher(256, 256, 256, 0)
    ref = O.ref_gemm(A, B)
    es = O.rel_frobenius(O.fused_fmm(A, B, *coeffs("strassen"), levels=1, blk=32), ref)
    ep = O.rel_frobenius(O.fused_fmm(A, B, *coeffs("phi_optimal"), levels=1, blk=32), ref)
    # Strassen's only error is the fp32 rounding of the scale amax/448 itself
    assert es < 2e-7 and ep > 1e-3


def test_gauge_invariance_of_rebalanced_coefficients():
    # App. E.2: the canonical rebalanced gauge cancels term by term (up to fp32 rounding of the factors)
    U, V, W = R.rebalanced(*R.winograd())
    U, V, W = (np.array(x, dtype=np.float32) for x in (U, V, W))
    A, B = Wl.gaussian(128, 128, 128, 9)
    ref = O.ref_gemm(A, B)
    e_raw = O.rel_frobenius(O.fused_fmm(A, B, *coeffs("winograd"), levels=1, blk=32), ref)
    e_bal = O.rel_frobenius(O.fused_fmm(A, B, U, V, W, levels=1, blk=32), ref)
    assert e_bal == pytest.approx(e_raw, rel=5e-3)


def test_error_stats_definition():
    rng = np.random.default_rng(0)
    C, Cr = rng.standard_normal((2, 50, 40))
    s = O.error_stats(C, Cr)
    assert s[0] == pytest.approx(((C - Cr) ** 2).sum(), rel=1e-14)
    assert s[1] == pytest.approx((Cr ** 2).sum(), rel=1e-14)
    assert s[2] == np.abs(C - Cr).max()
