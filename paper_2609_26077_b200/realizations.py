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


NAMED = {"strassen": strassen, "winograd": winograd, "phi_optimal": phi_optimal, "cubic8": cubic8}


def get(name):
    """fp32 (U, V, W) of a named realization."""
    U, V, W = NAMED[name]()
    return tuple(np.ascontiguousarray(x, dtype=np.float32) for x in (U, V, W))
