"""Exact coefficient algebra for rank-R 2x2 realizations (TEST INFRASTRUCTURE ONLY).

Part of the CPU oracle: exact arithmetic in Q(sqrt 3) for the realizations the
paper names, the Brent equations, and the coefficient functionals Phi and Gamma
(Sec. 2.1).  Nothing here is imported by the CUDA library or its Python binding.

Conventions (Sec. 2.1, App. A): a, b, c are the row vectorisations
(11, 12, 21, 22) of the 2x2 block matrices.  A realization is three R x 4 arrays
U, V, W with  c_q = sum_r <U_r, a> <V_r, b> W[r][q].  The paper's third factor is
the cyclic one, w_r = rv(W_r^T); `from_cyclic` converts it (swap entries 12 and 21).
"""
from __future__ import annotations

from fractions import Fraction as Fr
from itertools import product
import math


class Q3:
    """a + b*sqrt(3) with rational a, b."""
    __slots__ = ("a", "b")

    def __init__(self, a=0, b=0):
        self.a = Fr(a)
        self.b = Fr(b)

    @staticmethod
    def of(x):
        return x if isinstance(x, Q3) else Q3(x)

    def __add__(self, o):
        o = Q3.of(o)
        return Q3(self.a + o.a, self.b + o.b)

    __radd__ = __add__

    def __neg__(self):
        return Q3(-self.a, -self.b)

    def __sub__(self, o):
        return self + (-Q3.of(o))

    def __rsub__(self, o):
        return Q3.of(o) - self

    def __mul__(self, o):
        o = Q3.of(o)
        return Q3(self.a * o.a + 3 * self.b * o.b, self.a * o.b + self.b * o.a)

    __rmul__ = __mul__

    def __eq__(self, o):
        o = Q3.of(o)
        return self.a == o.a and self.b == o.b

    def __hash__(self):
        return hash((self.a, self.b))

    def is_zero(self):
        return self.a == 0 and self.b == 0

    def __float__(self):
        return float(self.a) + float(self.b) * math.sqrt(3.0)

    def __repr__(self):
        return f"({self.a}+{self.b}r3)"


SQRT3 = Q3(0, 1)
XI = Q3(0, Fr(1, 3))      # 1/sqrt(3)  = sqrt(3)/3
ETA = Q3(0, Fr(1, 2))     # sqrt(3)/2
ZETA = Q3(0, Fr(1, 6))    # 1/(2 sqrt 3) = sqrt(3)/6
H = Q3(Fr(1, 2))


def _rows(rows):
    return [[Q3.of(x) for x in r] for r in rows]


def strassen():
    """Strassen's seven products in the textbook order M1..M7."""
    U = _rows([(1, 0, 0, 1), (0, 0, 1, 1), (1, 0, 0, 0), (0, 0, 0, 1),
               (1, 1, 0, 0), (-1, 0, 1, 0), (0, 1, 0, -1)])
    V = _rows([(1, 0, 0, 1), (1, 0, 0, 0), (0, 1, 0, -1), (-1, 0, 1, 0),
               (0, 0, 0, 1), (1, 1, 0, 0), (0, 0, 1, 1)])
    W = _rows([(1, 0, 0, 1), (0, 0, 1, -1), (0, 1, 0, 1), (1, 0, 1, 0),
               (-1, 1, 0, 0), (0, 0, 0, 1), (1, 0, 0, 0)])
    return U, V, W


def winograd():
    """Flat coefficients of the 7-multiplication / 15-addition Strassen-Winograd variant."""
    U = _rows([(1, 0, 0, 0), (0, 1, 0, 0), (1, 1, -1, -1), (0, 0, 0, 1),
               (0, 0, 1, 1), (-1, 0, 1, 1), (1, 0, -1, 0)])
    V = _rows([(1, 0, 0, 0), (0, 0, 1, 0), (0, 0, 0, 1), (1, -1, -1, 1),
               (-1, 1, 0, 0), (1, -1, 0, 1), (0, -1, 0, 1)])
    W = _rows([(1, 1, 1, 1), (1, 0, 0, 0), (0, 1, 0, 0), (0, 0, -1, 0),
               (0, 1, 0, 1), (0, 1, 1, 1), (0, 0, 1, 1)])
    return U, V, W


def from_cyclic(w):
    """Paper's cyclic third factor w_r = rv(W_r^T)  ->  W[r][q] in the rv order of C."""
    return [[r[0], r[2], r[1], r[3]] for r in w]


def phi_optimal():
    """The certified Phi-minimiser T* from the printed coordinates (Eq. A.3):
    U* is printed; V*_r = U*_{pi_V(r)}; w*_r = U*_{pi_W(r)} in cyclic coordinates."""
    Us = _rows([(1, 0, 0, 1), (0, 0, XI, 1), (1, 0, XI, 0), (0, 0, -XI, 1),
                (H, ETA, ZETA, H), (-1, 0, XI, 0), (-H, ETA, ZETA, -H)])
    pi_v = (1, 3, 7, 6, 4, 5, 2)
    pi_w = (1, 7, 2, 5, 6, 4, 3)
    V = [list(Us[p - 1]) for p in pi_v]
    w = [list(Us[p - 1]) for p in pi_w]
    return Us, V, from_cyclic(w)


def cubic():
    """Rank-8 realization of the ordinary product: terms (i,j,k): a_ij * b_jk -> c_ik."""
    U, V, W = [], [], []
    for i, j, k in product(range(2), repeat=3):
        u = [Q3(0)] * 4
        v = [Q3(0)] * 4
        w = [Q3(0)] * 4
        u[2 * i + j] = Q3(1)
        v[2 * j + k] = Q3(1)
        w[2 * i + k] = Q3(1)
        U.append(u)
        V.append(v)
        W.append(w)
    return U, V, W


NAMED = {"strassen": strassen, "winograd": winograd, "phi_optimal": phi_optimal, "cubic": cubic}


def brent_residuals(U, V, W):
    """All 64 Brent equations for <2,2,2>:  for a = (i,j), b = (k,l), c = (m,n)
    sum_r U[r][a] V[r][b] W[r][c] = [j == k][i == m][l == n].  Returns the list of
    exact residuals (all zero iff the realization is an exact algorithm)."""
    res = []
    for i, j, k, l, m, n in product(range(2), repeat=6):
        s = Q3(0)
        for r in range(len(U)):
            s = s + Q3.of(U[r][2 * i + j]) * Q3.of(V[r][2 * k + l]) * Q3.of(W[r][2 * m + n])
        target = 1 if (j == k and i == m and l == n) else 0
        res.append(s - target)
    return res


def sqnorm(row):
    s = Q3(0)
    for x in row:
        s = s + Q3.of(x) * Q3.of(x)
    return s


def phi(U, V, W):
    """Phi(D) = sum_r |U_r|^2 |V_r|^2 |W_r|^2 (entrywise 2-norms), exact."""
    s = Q3(0)
    for r in range(len(U)):
        s = s + sqnorm(U[r]) * sqnorm(V[r]) * sqnorm(W[r])
    return s


def gamma(U, V, W):
    """Gamma(D) = sum_r |U_r| |V_r| |W_r| in floating point (needs square roots)."""
    return sum(math.sqrt(float(sqnorm(U[r])) * float(sqnorm(V[r])) * float(sqnorm(W[r])))
               for r in range(len(U)))


def kron(D1, D2):
    """Kronecker (recursive) composition: terms (r1, r2), coordinates (j1, j2)."""
    out = []
    for X1, X2 in zip(D1, D2):
        rows = []
        for r1 in X1:
            for r2 in X2:
                rows.append([Q3.of(a) * Q3.of(b) for a in r1 for b in r2])
        out.append(rows)
    return tuple(out)


def to_float(X):
    return [[float(x) for x in r] for r in X]


def rebalanced(U, V, W):
    """Canonical rebalanced gauge (App. E.2): (U_r/s_r, s_r V_r, W_r),
    s_r = sqrt(|U_r| / |V_r|); floating point."""
    Uo, Vo = [], []
    for r in range(len(U)):
        nu = math.sqrt(float(sqnorm(U[r])))
        nv = math.sqrt(float(sqnorm(V[r])))
        s = math.sqrt(nu / nv)
        Uo.append([float(x) / s for x in U[r]])
        Vo.append([float(x) * s for x in V[r]])
    return Uo, Vo, to_float(W)


def _inv_t(M):
    """Inverse transpose of a 2x2 matrix with rational (or float) entries."""
    (a, b), (c, d) = M
    det = a * d - b * c
    return [[d / det, -c / det], [-b / det, a / det]]


def _kron2(A, B):
    """4x4 Kronecker product of two 2x2 matrices, rows/columns in the rv order (11, 12, 21, 22)."""
    return [[A[i][j] * B[k][l] for j in range(2) for l in range(2)] for i in range(2) for k in range(2)]


def _rowmat(rows, M):
    return [[sum((r[j] * M[j][q] for j in range(4)), start=0 * r[0]) for q in range(4)] for r in rows]


def act(U, V, W, X, Y, Z):
    """Right action of (X, Y, Z) in GL_2^3 on a realization (Eq. A.1): u_r -> u_r (X (x) Y^-T),
    v_r -> v_r (Y (x) Z^-T), w_r -> w_r (Z (x) X^-T) on the cyclic third factor.  Exact when the
    coefficients are Q3 and the matrices hold Fractions; floating point otherwise."""
    w = from_cyclic(W)          # the swap of entries 12 and 21 is its own inverse
    return (_rowmat(U, _kron2(X, _inv_t(Y))), _rowmat(V, _kron2(Y, _inv_t(Z))),
            from_cyclic(_rowmat(w, _kron2(Z, _inv_t(X)))))


class _Jet:
    """c0 + c1 s + c2 s^2 (higher powers of s dropped), coefficients in Q(sqrt 3)."""
    __slots__ = ("c",)

    def __init__(self, c0=0, c1=0, c2=0):
        self.c = (Q3.of(c0), Q3.of(c1), Q3.of(c2))

    @staticmethod
    def of(x):
        return x if isinstance(x, _Jet) else _Jet(x)

    def __add__(self, o):
        o = _Jet.of(o)
        return _Jet(*(a + b for a, b in zip(self.c, o.c)))

    __radd__ = __add__

    def __mul__(self, o):
        o = _Jet.of(o)
        a, b = self.c, o.c
        return _Jet(a[0] * b[0], a[0] * b[1] + a[1] * b[0], a[0] * b[2] + a[1] * b[1] + a[2] * b[0])

    __rmul__ = __mul__


def phi_second_order(U, V, W, direction):
    """Exact coefficient of s^2 in Phi(D . (e^{s H_X}, e^{s H_Y}, e^{s H_Z})) (App. A, second-order form),
    with direction = (x1, y1, z1, x2, y2, z2) rational and H(p, q) = 1/2 [[p, q], [q, -p]].
    H is symmetric, so e^{sH} = I + sH + s^2 H^2 / 2 + ... and (e^{sH})^-T = e^{-sH}; terms beyond s^2
    cannot reach the coefficient, which makes a truncated series exact."""
    x1, y1, z1, x2, y2, z2 = (Fr(d) for d in direction)

    def expo(p, q, sign):
        h = [[p / 2, q / 2], [q / 2, -p / 2]]
        h2 = [[sum(h[i][k] * h[k][j] for k in range(2)) for j in range(2)] for i in range(2)]
        return [[_Jet(1 if i == j else 0, sign * h[i][j], h2[i][j] / 2) for j in range(2)] for i in range(2)]

    X, Xi = expo(x1, x2, 1), expo(x1, x2, -1)
    Y, Yi = expo(y1, y2, 1), expo(y1, y2, -1)
    Z, Zi = expo(z1, z2, 1), expo(z1, z2, -1)

    def kron(A, B):
        return [[A[i][j] * B[k][l] for j in range(2) for l in range(2)] for i in range(2) for k in range(2)]

    def rows_times(rows, M):
        out = []
        for r in rows:
            out.append([sum((_Jet.of(r[j]) * M[j][q] for j in range(4)), _Jet()) for q in range(4)])
        return out

    def sq(row):
        return sum((x * x for x in row), _Jet())

    U2 = rows_times(U, kron(X, Yi))
    V2 = rows_times(V, kron(Y, Zi))
    w2 = rows_times(from_cyclic(W), kron(Z, Xi))        # squared row norms do not depend on the entry order
    total = _Jet()
    for r in range(len(U)):
        total = total + sq(U2[r]) * sq(V2[r]) * sq(w2[r])
    return total.c


def phi_hessian(U, V, W):
    """6 x 6 matrix of second derivatives of Phi at the realization in the coordinates t of App. A
    (exact, by polarization of phi_second_order): Phi_t = Phi + g.t + 1/2 t^T Hess t + O(|t|^3)."""
    e = [[1 if i == j else 0 for j in range(6)] for i in range(6)]
    diag = [phi_second_order(U, V, W, e[i])[2] for i in range(6)]
    Hs = [[None] * 6 for _ in range(6)]
    for i in range(6):
        Hs[i][i] = diag[i] * 2
        for j in range(i + 1, 6):
            both = phi_second_order(U, V, W, [e[i][k] + e[j][k] for k in range(6)])[2]
            Hs[i][j] = Hs[j][i] = both - diag[i] - diag[j]
    return Hs
