"""Pins for the oracle's coefficient algebra: exact Brent equations, Phi / Gamma values the
paper prints, the printed coordinates of the certified optimum, and the 5/3 floor."""
from fractions import Fraction as Fr
import math

import numpy as np
import pytest

from oracle import realizations as R
from oracle.realizations import Q3, XI, ETA


@pytest.mark.parametrize("name", ["strassen", "winograd", "phi_optimal", "cubic"])
def test_brent_equations_exact(name):
    U, V, W = R.NAMED[name]()
    res = R.brent_residuals(U, V, W)
    assert len(res) == 64
    assert all(x.is_zero() for x in res)


def test_brent_detects_wrong_w_convention():
    # using the paper's cyclic third factor untransposed is NOT an exact algorithm
    U, V, W = R.phi_optimal()
    w_cyclic = R.from_cyclic(W)          # involution: back to cyclic coordinates
    bad = [x for x in R.brent_residuals(U, V, w_cyclic) if not x.is_zero()]
    assert len(bad) > 0


def test_phi_values_exact():
    # Sec. 3 / Table E.2: cubic 8, Strassen 32, Winograd form 56, certified optimum 200/9
    assert R.phi(*R.cubic()) == Q3(8)
    assert R.phi(*R.strassen()) == Q3(32)
    assert R.phi(*R.winograd()) == Q3(56)
    assert R.phi(*R.phi_optimal()) == Q3(Fr(200, 9))


def test_gamma_values():
    # Table E.2 and App. C
    from golden_values import figures, panel
    tab = panel()                    # Table E.2 as printed (tests/golden/table_e2_panel.tsv)
    assert R.gamma(*R.strassen()) == pytest.approx(tab["strassen_classic"][2], abs=5e-5)
    assert R.gamma(*R.winograd()) == pytest.approx(tab["winograd_form"][2], abs=5e-5)
    assert R.gamma(*R.phi_optimal()) == pytest.approx(tab["dps_acc"][2], abs=5e-5)
    assert R.gamma(*R.phi_optimal()) == pytest.approx(figures()["gamma_optimal_exact"], abs=1e-11)
    assert float(R.phi(*R.strassen()).a) == tab["strassen_classic"][1] and float(R.phi(*R.winograd()).a) == tab["winograd_form"][1]
    assert float(R.phi(*R.phi_optimal()).a) == pytest.approx(tab["dps_acc"][1], abs=5e-5)
    assert R.gamma(*R.phi_optimal()) == pytest.approx(2 * math.sqrt(2) + 16 / math.sqrt(3), abs=1e-12)


def test_optimum_row_norms():
    # Eq. (A.4): squared row norms (2, 4/3 x 6) for each of U*, V*, W*
    want = [Q3(2)] + [Q3(Fr(4, 3))] * 6
    for X in R.phi_optimal():
        assert [R.sqnorm(r) for r in X] == want


def test_optimum_is_strassen_times_k_rho():
    # App. A: U* = U_Strassen * K_rho with K_rho = T_rho (x) T_rho^-T, rho^2 = 2/sqrt 3
    rho2, rho_m2 = 2 * XI, ETA
    K = [[Q3(1), Q3(0), rho2 * Fr(1, 2), Q3(0)],
         [Q3(Fr(-1, 2)), rho_m2, rho2 * Fr(-1, 4), Q3(Fr(1, 2))],
         [Q3(0), Q3(0), rho2, Q3(0)],
         [Q3(0), Q3(0), rho2 * Fr(-1, 2), Q3(1)]]
    Us = R.strassen()[0]
    got = [[sum((Us[r][i] * K[i][j] for i in range(4)), Q3(0)) for j in range(4)] for r in range(7)]
    assert got == R.phi_optimal()[0]


def _mat(row):
    return [[row[0], row[1]], [row[2], row[3]]]


def _mm(A, B):
    return [[sum((A[i][k] * B[k][j] for k in range(2)), Q3(0)) for j in range(2)] for i in range(2)]


def _tr(A):
    return [[A[0][0], A[1][0]], [A[0][1], A[1][1]]]


def test_moment_map_isotropy():
    # App. A: L_A = sum a_r^2 A_r A_r^T = (100/9) I and R_A likewise, for A = U*, V*, w*
    U, V, W = R.phi_optimal()
    w = R.from_cyclic(W)
    for X in (U, V, w):
        L = [[Q3(0)] * 2 for _ in range(2)]
        Rr = [[Q3(0)] * 2 for _ in range(2)]
        for row in X:
            a2 = R.sqnorm(row) * R.sqnorm(row)
            A = _mat(row)
            AAt, AtA = _mm(A, _tr(A)), _mm(_tr(A), A)
            for i in range(2):
                for j in range(2):
                    L[i][j] = L[i][j] + a2 * AAt[i][j]
                    Rr[i][j] = Rr[i][j] + a2 * AtA[i][j]
        iso = [[Q3(Fr(100, 9)), Q3(0)], [Q3(0), Q3(Fr(100, 9))]]
        assert L == iso and Rr == iso


def _act(D, X, Y, Z):
    """Right action of Eq. (A.1) in cyclic coordinates (floating point)."""
    U, V, W = [np.array(R.to_float(x)) for x in D]
    w = W[:, [0, 2, 1, 3]]
    inv_t = lambda M: np.linalg.inv(M).T
    U2 = U @ np.kron(X, inv_t(Y))
    V2 = V @ np.kron(Y, inv_t(Z))
    w2 = w @ np.kron(Z, inv_t(X))
    return U2, V2, w2[:, [0, 2, 1, 3]]


def _phi_f(U, V, W):
    return float(np.sum((U ** 2).sum(1) * (V ** 2).sum(1) * (W ** 2).sum(1)))


def _brent_f(U, V, W):
    T = np.einsum("ra,rb,rc->abc", U, V, W)
    want = np.zeros((4, 4, 4))
    for i in range(2):
        for j in range(2):
            for l in range(2):
                want[2 * i + j, 2 * j + l, 2 * i + l] = 1
    return np.abs(T - want).max()


def test_sandwich_reaches_optimum_and_floor_holds():
    # Strassen sandwiched by X = Y = Z = T_rho lands on Phi = 200/9 (Thm 1), the action keeps
    # exactness, and no sampled point of the orbit goes below the floor: sqrt(Phi/8) >= 5/3.
    rho = (4.0 / 3.0) ** 0.25
    T = np.array([[1 / rho, rho / 2], [0, rho]])
    D = _act(R.strassen(), T, T, T)
    assert _brent_f(*D) < 1e-12
    assert _phi_f(*D) == pytest.approx(200 / 9, rel=1e-12)
    np.testing.assert_allclose(D[0], np.array(R.to_float(R.phi_optimal()[0])), atol=1e-12)
    rng = np.random.default_rng(1)
    for trial in range(200):
        scale = [0.02, 0.2, 0.45][trial % 3]
        X, Y, Z = (np.eye(2) + scale * rng.standard_normal((2, 2)) for _ in range(3))
        if min(abs(np.linalg.det(M)) for M in (X, Y, Z)) < 1e-3:
            continue
        Dg = _act(R.phi_optimal(), X, Y, Z)
        assert _brent_f(*Dg) < 1e-9
        assert _phi_f(*Dg) >= 200 / 9 - 1e-9
    for name in ("strassen", "winograd", "phi_optimal"):
        ratio = math.sqrt(float(R.phi(*R.NAMED[name]())) / 8.0)
        assert ratio >= 5 / 3 - 1e-15
    assert math.sqrt(float(R.phi(*R.phi_optimal())) / 8.0) == pytest.approx(5 / 3, rel=1e-15)
    assert math.sqrt(32 / 8) == 2 and math.sqrt(56 / 8) == pytest.approx(math.sqrt(7))


def test_phi_multiplicative_under_kronecker():
    # Sec. 3: Phi(D (x) D) = Phi(D)^2, and the Kronecker square is an exact <4,4,4;49> algorithm
    for name in ("strassen", "phi_optimal"):
        D = R.NAMED[name]()
        D2 = R.kron(D, D)
        assert len(D2[0]) == 49
        assert R.phi(*D2) == R.phi(*D) * R.phi(*D)


def test_winograd_rebalance_factors():
    # App. E.5: exactly two Winograd terms get rebalancing factors sqrt 2 and 1/sqrt 2
    U, V, W = R.winograd()
    s = [math.sqrt(math.sqrt(float(R.sqnorm(U[r])) / float(R.sqnorm(V[r])))) for r in range(7)]
    off = sorted(x for x in s if abs(x - 1) > 1e-12)
    assert off == pytest.approx([1 / math.sqrt(2), math.sqrt(2)])


def test_second_order_form_and_hessian_spectrum_at_the_optimum():
    # App. A, second-order form: Phi_t = 200/9 + (8/9) t^T diag(Q, Q) t + O(|t|^3) with the printed Q; the
    # coordinate Hessian has eigenvalues 128/9 (twice) and 440/9 (four times).  All in exact arithmetic.
    U, V, W = R.phi_optimal()
    Qm = [[Fr(21), Fr(-13, 2), Fr(-13, 2)], [Fr(-13, 2), Fr(21), Fr(-13, 2)], [Fr(-13, 2), Fr(-13, 2), Fr(21)]]
    Hs = R.phi_hessian(U, V, W)
    for i in range(6):
        for j in range(6):
            same_block = (i // 3) == (j // 3)
            want = Fr(16, 9) * Qm[i % 3][j % 3] if same_block else Fr(0)
            assert Hs[i][j] == Q3(want), (i, j, Hs[i][j])
    # stationarity (zero moment map): no first-order term in any coordinate or pair direction
    for d in ([1, 0, 0, 0, 0, 0], [0, 0, 0, 0, 1, 0], [1, -2, 3, 5, -1, 2]):
        c0, c1, _ = R.phi_second_order(U, V, W, d)
        assert c0 == Q3(Fr(200, 9)) and c1.is_zero()
    # spectrum: (H - 128/9)(H - 440/9) = 0 with trace 2 * 128/9 + 4 * 440/9, so exactly those multiplicities
    lo, hi = Fr(128, 9), Fr(440, 9)
    Hf = [[Hs[i][j].a for j in range(6)] for i in range(6)]
    A1 = [[Hf[i][j] - (lo if i == j else 0) for j in range(6)] for i in range(6)]
    A2 = [[Hf[i][j] - (hi if i == j else 0) for j in range(6)] for i in range(6)]
    prod = [[sum(A1[i][k] * A2[k][j] for k in range(6)) for j in range(6)] for i in range(6)]
    assert all(x == 0 for row in prod for x in row)
    assert sum(Hf[i][i] for i in range(6)) == 2 * lo + 4 * hi
    assert np.allclose(np.sort(np.linalg.eigvalsh(np.array(Hf, dtype=float))),
                       [128 / 9] * 2 + [440 / 9] * 4, rtol=1e-12)
    # control: classic Strassen is not a stationary point of Phi on its orbit
    c0, c1, _ = R.phi_second_order(*R.strassen(), [0, 0, 0, 1, 0, 0])
    assert c0 == Q3(32) and not c1.is_zero()
