"""fp32 coefficient tables of the named rank-7 realizations of 2x2 matrix multiplication
(Sec. 2.1; Sec. 3 / App. A for the Phi-optimal one), in this library's convention:
rows = terms, columns = blocks 11, 12, 21, 22, and W[r][q] = weight of product r in C_q.
"""
from __future__ import annotations

import math

import numpy as np


def _arr(rows):
    return np.array(rows, dtype=np.float64)


def strassen():
    """Strassen's original seven products (Phi = 32)."""
    U = _arr([[1, 0, 0, 1], [0, 0, 1, 1], [1, 0, 0, 0], [0, 0, 0, 1], [1, 1, 0, 0], [-1, 0, 1, 0], [0, 1, 0, -1]])
    V = _arr([[1, 0, 0, 1], [1, 0, 0, 0], [0, 1, 0, -1], [-1, 0, 1, 0], [0, 0, 0, 1], [1, 1, 0, 0], [0, 0, 1, 1]])
    W = _arr([[1, 0, 0, 1], [0, 0, 1, -1], [0, 1, 0, 1], [1, 0, 1, 0], [-1, 1, 0, 0], [0, 0, 0, 1], [1, 0, 0, 0]])
    return U, V, W


def winograd():
    """Flat coefficients of the Strassen-Winograd variant (Phi = 56)."""
    U = _arr([[1, 0, 0, 0], [0, 1, 0, 0], [1, 1, -1, -1], [0, 0, 0, 1], [0, 0, 1, 1], [-1, 0, 1, 1], [1, 0, -1, 0]])
    V = _arr([[1, 0, 0, 0], [0, 0, 1, 0], [0, 0, 0, 1], [1, -1, -1, 1], [-1, 1, 0, 0], [1, -1, 0, 1], [0, -1, 0, 1]])
    W = _arr([[1, 1, 1, 1], [1, 0, 0, 0], [0, 1, 0, 0], [0, 0, -1, 0], [0, 1, 0, 1], [0, 1, 1, 1], [0, 0, 1, 1]])
    return U, V, W


def phi_optimal():
    """The certified Phi-minimiser (Phi = 200/9): Strassen sandwiched by X = Y = Z = T_rho,
    rho = (4/3)^(1/4) (App. A).  Built from the sandwich action rather than typed in:
    u_r -> u_r (X (x) Y^-T), v_r -> v_r (Y (x) Z^-T), w_r -> w_r (Z (x) X^-T) on the cyclic third factor."""
    rho = (4.0 / 3.0) ** 0.25
    T = np.array([[1.0 / rho, rho / 2.0], [0.0, rho]])
    Tit = np.linalg.inv(T).T
    K = np.kron(T, Tit)
    U, V, W = strassen()
    w = W[:, [0, 2, 1, 3]]
    U2, V2, w2 = U @ K, V @ K, w @ K
    return _clean(U2), _clean(V2), _clean(w2[:, [0, 2, 1, 3]])


def _clean(X):
    X = X.copy()
    X[np.abs(X) < 1e-14] = 0.0
    return X


def cubic8():
    """Rank-8 realization of the ordinary product (Phi = 8)."""
    U = np.zeros((8, 4)); V = np.zeros((8, 4)); W = np.zeros((8, 4))
    r = 0
    for i in range(2):
        for j in range(2):
            for k in range(2):
                U[r, 2 * i + j] = 1; V[r, 2 * j + k] = 1; W[r, 2 * i + k] = 1
                r += 1
    return U, V, W


def rebalanced(U, V, W):
    """Canonical rebalanced gauge of App. E.2: (U_r / s_r, s_r V_r, W_r), s_r = sqrt(|U_r| / |V_r|)."""
    s = np.sqrt(np.linalg.norm(U, axis=1) / np.linalg.norm(V, axis=1))
    return U / s[:, None], V * s[:, None], W.copy()


def phi(U, V, W):
    """Phi = sum_r |U_r|^2 |V_r|^2 |W_r|^2 (Sec. 2.1)."""
    U, V, W = (np.asarray(x, dtype=np.float64) for x in (U, V, W))
    return float(np.sum((U ** 2).sum(1) * (V ** 2).sum(1) * (W ** 2).sum(1)))


def act(U, V, W, X, Y, Z):
    """Right action of g = (X, Y, Z) in GL_2^3 on a realization (Eq. A.1):
    u_r -> u_r (X (x) Y^-T), v_r -> v_r (Y (x) Z^-T), w_r -> w_r (Z (x) X^-T), with w_r the cyclic third
    factor rv(W_r^T), i.e. this library's W row with entries 12 and 21 swapped."""
    it = lambda M: np.linalg.inv(M).T
    cyc = [0, 2, 1, 3]
    U2 = np.asarray(U, dtype=np.float64) @ np.kron(X, it(Y))
    V2 = np.asarray(V, dtype=np.float64) @ np.kron(Y, it(Z))
    w2 = np.asarray(W, dtype=np.float64)[:, cyc] @ np.kron(Z, it(X))
    return U2, V2, w2[:, cyc]


_DIRECTIONS = {"diag": np.array([[1.0, 0.0], [0.0, -1.0]]), "shear": np.array([[0.0, 1.0], [1.0, 0.0]])}


def orbit_perturbation(factor, direction, sign, phi_target=24.0):
    """A local perturbation of the Phi-optimal realization along one geodesic of the orbit (App. E.4):
    T* . g with g = exp(sign * delta * H) in factor `factor` (0, 1, 2 = X, Y, Z), H = diag(1, -1) ("diag")
    or [[0, 1], [1, 0]] ("shear"), and delta > 0 solved so that Phi = phi_target.  Phi is convex along the
    geodesic with its minimum 200/9 at delta = 0 (Eq. A.2), so bisection on delta is enough.
    Returns (U, V, W, delta) in float64, raw gauge."""
    U, V, W = phi_optimal()
    ev, Q = np.linalg.eigh(_DIRECTIONS[direction])

    def arm(delta):
        g = [np.eye(2), np.eye(2), np.eye(2)]
        g[factor] = Q @ np.diag(np.exp(sign * delta * ev)) @ Q.T
        return act(U, V, W, *g)

    lo, hi = 0.0, 1.0
    while phi(*arm(hi)) < phi_target:
        hi *= 2.0
    for _ in range(100):
        mid = 0.5 * (lo + hi)
        if phi(*arm(mid)) < phi_target:
            lo = mid
        else:
            hi = mid
    delta = 0.5 * (lo + hi)
    return (*arm(delta), delta)


def orbit_member(k, spread=0.25):
    """Member k of a seeded family of exact orbit points T* . g_k (App. E.8, orbit-ratio stability): in each
    factor g = exp(S) R with S a random symmetric traceless matrix of norm <= spread and R a random rotation,
    so the members differ in Phi as well as in frame.  Member 0 is T* itself."""
    U, V, W = phi_optimal()
    if k == 0:
        return U, V, W
    rng = np.random.default_rng([2609, 26077, k])
    g = []
    for _ in range(3):
        a, b = rng.uniform(-spread, spread, 2) / math.sqrt(2.0)
        ev, Q = np.linalg.eigh(np.array([[a, b], [b, -a]]))
        th = rng.uniform(0.0, 2.0 * math.pi)
        R = np.array([[math.cos(th), -math.sin(th)], [math.sin(th), math.cos(th)]])
        g.append(Q @ np.diag(np.exp(ev)) @ Q.T @ R)
    return act(U, V, W, *g)


NAMED = {"strassen": strassen, "winograd": winograd, "phi_optimal": phi_optimal, "cubic8": cubic8}
PERTURBATIONS = [f"pert_f{f}_{d}_{s}" for f in range(3) for d in ("diag", "shear") for s in ("p", "m")]
# the reconstructible part of the paper's fixed panel (Table E.2): three named arms and the twelve signed
# perturbations at Phi = 24, all in the rebalanced gauge
ORBIT15 = [f"orbit_{k:02d}_rb" for k in range(15)]
LADDER = ["phi_optimal_rb"] + [n + "_rb" for n in PERTURBATIONS] + ["strassen_rb", "winograd_rb"]


def get64(name):
    """float64 (U, V, W) of a named realization; `<name>_rb` = the same in the rebalanced gauge;
    `pert_f<0|1|2>_<diag|shear>_<p|m>` = orbit_perturbation at Phi = 24; `orbit_<k>` = orbit_member(k)."""
    if name.endswith("_rb"):
        return rebalanced(*get64(name[:-3]))
    if name.startswith("pert_"):
        _, f, d, s = name.split("_")
        return orbit_perturbation(int(f[1]), d, +1 if s == "p" else -1)[:3]
    if name.startswith("orbit_"):
        return orbit_member(int(name.split("_")[1]))
    return NAMED[name]()


def get(name):
    """fp32 (U, V, W) of a named realization (see get64 for the names)."""
    return tuple(np.ascontiguousarray(x, dtype=np.float32) for x in get64(name))
