"""CPU checks of the boundary: the C-ABI library loads, exports every declared symbol, and its
host-side logic (validation, Phi/Gamma, Brent residual) behaves; no compute calls without a GPU."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2609_26077_b200 import build as fmm_build
from paper_2609_26077_b200 import fmm, realizations as P

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fmm_build.build()
    return fmm.lib()


def test_every_declared_symbol_is_exported(lib):
    text = open(os.path.join(ROOT, "include", "fmm.h")).read()
    declared = set(re.findall(r"\b(fmm_[a-z0-9_]+)\s*\(", text))
    declared -= {"fmm_plan"}
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in fmm.h but not exported"
    assert declared == set(fmm.EXPORTS)


def test_phi_gamma_and_brent_host_utilities(lib):
    phi, gam = fmm.fmm_phi_gamma(*P.get("strassen"))
    assert phi == 32.0 and gam == pytest.approx(14.828427, abs=1e-6)
    phi, gam = fmm.fmm_phi_gamma(*P.get("winograd"))
    assert phi == 56.0 and gam == pytest.approx(17.853007, abs=1e-6)
    phi, gam = fmm.fmm_phi_gamma(*P.get("phi_optimal"))
    assert phi == pytest.approx(200 / 9, rel=1e-6) and gam == pytest.approx(12.0660314, rel=1e-6)
    assert fmm.fmm_phi_gamma(*P.get("cubic8"))[0] == 8.0
    for name in P.NAMED:
        assert fmm.fmm_brent_residual(*P.get(name)) < 1e-6
    U, V, W = P.get("strassen")
    W = W.copy(); W[0, 1] = 0.41
    assert fmm.fmm_brent_residual(U, V, W) == pytest.approx(0.41, rel=1e-6)


def test_plan_create_rejects_bad_arguments(lib):
    U, V, W = P.get("strassen")
    qp = fmm.QuantParams(32, 0, 1e-12, 448.0)
    h = C.c_void_p()
    f = lambda a: a.ctypes.data_as(C.POINTER(C.c_float))
    call = lambda rank, u, v, w, levels, q: lib.fmm_plan_create(C.byref(h), rank, u, v, w, levels, C.byref(q) if q else None)
    assert call(7, f(U), f(V), f(W), 4, qp) == 1                      # levels out of range
    assert call(9, f(U), f(V), f(W), 1, qp) == 1                      # rank out of range
    assert call(7, None, f(V), f(W), 1, qp) == 1                      # null coefficients
    assert call(7, f(U), f(V), f(W), 1, None) == 1
    assert call(7, f(U), f(V), f(W), 1, fmm.QuantParams(64, 0, 1e-12, 448.0)) == 1    # block size
    assert call(7, f(U), f(V), f(W), 1, fmm.QuantParams(128, 1, 1e-12, 448.0)) == 1   # UE8M0 needs 32
    assert call(7, f(U), f(V), f(W), 1, fmm.QuantParams(32, 0, 1e-12, 240.0)) == 1    # not e4m3's max
    Wbad = W.copy(); Wbad[3, 2] = -1.0
    assert call(7, f(U), f(V), f(Wbad), 1, qp) == 3                   # FMM_ERR_NOT_EXACT
    wc = np.ascontiguousarray(P.get("phi_optimal")[2][:, [0, 2, 1, 3]])  # cyclic third factor, untransposed
    Uo, Vo, _ = P.get("phi_optimal")
    assert call(7, f(Uo), f(Vo), f(wc), 1, qp) == 3
    assert lib.fmm_plan_create(None, 7, f(U), f(V), f(W), 1, C.byref(qp)) == 1
    assert lib.fmm_plan_destroy(None) == 1
    # without a CUDA device a valid request fails loudly instead of falling back
    import torch
    if not torch.cuda.is_available():
        assert call(7, f(U), f(V), f(W), 1, qp) in (6, 7)
        with pytest.raises(fmm.FmmError):
            fmm.Plan(U, V, W)


def test_status_strings(lib):
    for s in range(9):
        assert lib.fmm_status_string(s)
    assert lib.fmm_error_stats_scratch_bytes() >= 3 * 8
