"""The orbit action (Eq. A.1) and the reconstructible part of the paper's fixed panel (Table E.2):
pins for the oracle's exact action and for the perturbation arms the package generates."""
import math
from fractions import Fraction as Fr

import numpy as np
import pytest

from oracle import realizations as R
from paper_2609_26077_b200 import realizations as P


def _exact_zero(res):
    return all(x.is_zero() for x in res)


def test_action_preserves_brent_equations_exactly():
    # any g in GL_2(Q)^3 maps an exact algorithm to an exact algorithm; a wrong slot, a missing inverse or
    # a missing transpose in Eq. (A.1) breaks at least one of the 64 equations
    X = [[Fr(2), Fr(1)], [Fr(1), Fr(1)]]
    Y = [[Fr(1), Fr(-3)], [Fr(0), Fr(2)]]
    Z = [[Fr(1, 2), Fr(0)], [Fr(5), Fr(3)]]
    for name in ("strassen", "winograd", "phi_optimal"):
        U, V, W = R.act(*R.NAMED[name](), X, Y, Z)
        assert _exact_zero(R.brent_residuals(U, V, W)), name


def test_phi_is_invariant_under_rotations_exactly():
    # O(2)^3 preserves Phi (App. A); rational rotation with (3/5, 4/5) and a reflection
    Q = [[Fr(3, 5), Fr(-4, 5)], [Fr(4, 5), Fr(3, 5)]]
    Fm = [[Fr(0), Fr(1)], [Fr(1), Fr(0)]]
    I = [[Fr(1), Fr(0)], [Fr(0), Fr(1)]]
    for g in ((Q, I, I), (I, Q, Fm), (Q, Fm, Q)):
        U, V, W = R.act(*R.phi_optimal(), *g)
        assert R.phi(U, V, W) == R.Q3(Fr(200, 9))
        assert _exact_zero(R.brent_residuals(U, V, W))


def test_scalar_gauge_moves_phi_nowhere_but_diag_scaling_does():
    # central scalars act by (s_X/s_Y, s_Y/s_Z, s_Z/s_X), product one: Phi unchanged
    s = lambda a: [[Fr(a), Fr(0)], [Fr(0), Fr(a)]]
    U, V, W = R.act(*R.strassen(), s(2), s(3), s(5))
    assert R.phi(U, V, W) == R.Q3(32)
    # a genuine diagonal element changes Phi of Strassen's algorithm
    D = [[Fr(2), Fr(0)], [Fr(0), Fr(1, 2)]]
    I = s(1)
    U, V, W = R.act(*R.strassen(), D, I, I)
    assert R.phi(U, V, W) != R.Q3(32)


def test_package_action_agrees_with_exact_action():
    X = np.array([[2.0, 1.0], [1.0, 1.0]]); Y = np.array([[1.0, -3.0], [0.0, 2.0]]); Z = np.array([[0.5, 0.0], [5.0, 3.0]])
    fr = lambda M: [[Fr(x).limit_denominator(1000) for x in r] for r in M.tolist()]
    want = [np.array(R.to_float(x)) for x in R.act(*R.strassen(), fr(X), fr(Y), fr(Z))]
    got = P.act(*P.strassen(), X, Y, Z)
    for g, w in zip(got, want):
        assert np.allclose(g, w, rtol=0, atol=1e-12)


@pytest.mark.parametrize("name", P.PERTURBATIONS)
def test_perturbation_arms_are_exact_algorithms_at_phi_24(name):
    U, V, W = P.get64(name)
    res = R.brent_residuals(*[[[float(x) for x in r] for r in M] for M in (U, V, W)])
    assert max(abs(float(x)) for x in res) < 1e-12
    assert abs(P.phi(U, V, W) - 24.0) < 1e-9
    # rebalanced gauge: equal encoder norms in every term, Phi and Gamma unchanged
    Ur, Vr, Wr = P.get64(name + "_rb")
    assert np.allclose(np.linalg.norm(Ur, axis=1), np.linalg.norm(Vr, axis=1), rtol=1e-12)
    assert abs(P.phi(Ur, Vr, Wr) - 24.0) < 1e-9


def test_phi_along_a_geodesic_has_the_kempf_ness_form():
    # Eq. (A.2): F(t) = sum_lambda e^{2 lambda t} |w_lambda|^2.  A one-factor direction H with eigenvalues +-1
    # enters two of the three tensor slots, so lambda is in {-2, 0, 2}; at the minimiser the +-2 weights are
    # equal and F(t) = b + 2a cosh(4t): symmetric in t, and (F(t) - F(0)) / (cosh 4t - 1) is constant.
    U, V, W = P.phi_optimal()
    for factor in range(3):
        for H in (np.array([[1.0, 0.0], [0.0, -1.0]]), np.array([[0.0, 1.0], [1.0, 0.0]])):
            ev, Q = np.linalg.eigh(H)
            vals = []
            for t in (0.05, 0.1, 0.2, 0.4):
                f = []
                for sgn in (1, -1):
                    g = [np.eye(2)] * 3
                    g[factor] = Q @ np.diag(np.exp(sgn * t * ev)) @ Q.T
                    f.append(P.phi(*P.act(U, V, W, *g)))
                assert abs(f[0] - f[1]) < 1e-10
                vals.append((f[0] - 200.0 / 9.0) / (math.cosh(4 * t) - 1.0))
            assert max(vals) - min(vals) < 1e-9
            # 2a = 28/3 here, hence cosh(4 delta) = 1 + (24 - 200/9) / (28/3) = 25/21 at Phi = 24
            assert abs(vals[0] - 28.0 / 3.0) < 1e-9
    for name in P.PERTURBATIONS:
        _, f, d, s = name.split("_")
        delta = P.orbit_perturbation(int(f[1]), d, +1 if s == "p" else -1)[3]
        assert abs(delta - math.acosh(25.0 / 21.0) / 4.0) < 1e-9


def test_gamma_values_against_the_printed_panel():
    # Table E.2 prints Gamma = sum_r |U_r||V_r||W_r| for every arm: 12.0660 for the optimum, 14.8284 for
    # Strassen, 17.8530 for the Winograd form, and, for the twelve Phi = 24 arms, 12.4549 / 12.4791 (six arms)
    # and values between 12.4658 and 12.4683 (six arms).  The artifact's coordinate frame is not printed, so
    # arm labels cannot be matched one to one; the two families of values can.
    from golden_values import panel
    tab = panel()                    # tests/golden/table_e2_panel.tsv
    g = lambda n: R.gamma(*[[[float(x) for x in r] for r in M] for M in P.get64(n)])
    assert round(g("phi_optimal"), 4) == tab["dps_acc"][2]
    assert round(g("strassen"), 4) == tab["strassen_classic"][2]
    assert round(g("winograd"), 4) == tab["winograd_form"][2]
    printed = sorted(v[2] for k, v in tab.items() if v[0] == "P")
    assert all(v[1] == 24.0 for v in tab.values() if v[0] == "P") and len(printed) == 12
    # the printed values fall into two families: three arms each at the two extremes, six in between
    lo, hi = printed[0], printed[-1]
    assert printed[:3] == [lo] * 3 and printed[-3:] == [hi] * 3
    extreme = sorted(round(g(n), 4) for n in P.PERTURBATIONS if "_diag_" in n)
    assert extreme == [lo] * 3 + [hi] * 3
    for n in P.PERTURBATIONS:
        if "_shear_" in n:
            assert printed[3] - 0.0015 < g(n) < printed[8] + 0.0015
        assert abs(g(n) - g(n + "_rb")) < 1e-12       # Gamma does not see the gauge


def test_ladder_is_ordered_by_phi():
    phis = [P.phi(*P.get64(n)) for n in P.LADDER]
    assert all(b >= a - 1e-9 for a, b in zip(phis, phis[1:]))
    assert abs(phis[0] - 200.0 / 9.0) < 1e-12 and abs(phis[-2] - 32.0) < 1e-12 and abs(phis[-1] - 56.0) < 1e-12


def test_orbit_members_are_exact_algorithms_with_phi_above_the_minimum():
    # every member of the orbit satisfies the Brent equations and has Phi >= 200/9 (the certificate, Sec. 3)
    phis = []
    for name in P.ORBIT15:
        U, V, W = P.get64(name)
        res = R.brent_residuals(*[[[float(x) for x in r] for r in M] for M in (U, V, W)])
        assert max(abs(float(x)) for x in res) < 1e-12
        phis.append(P.phi(U, V, W))
    assert abs(phis[0] - 200.0 / 9.0) < 1e-12
    assert all(p > 200.0 / 9.0 + 1e-6 for p in phis[1:])
    assert max(phis) > 28.0          # the family spans a range of Phi, not just frames
