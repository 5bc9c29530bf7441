"""The library's own fp32 coefficient tables against the oracle's exact ones.

The two sides build the named realizations independently: the oracle types the printed coordinates (Eq. A.3 for the
certified optimum, with the permutations pi_V, pi_W and the cyclic third factor) in Q(sqrt 3); the library derives
the optimum from the sandwich action on Strassen in float64.  Every GPU parity test hands the library's tables to
both sides, so the tables themselves are pinned here, bit for bit in fp32."""
import numpy as np
import pytest

from oracle import realizations as R
from paper_2609_26077_b200 import realizations as P


@pytest.mark.parametrize("lib_name,oracle_name", [("strassen", "strassen"), ("winograd", "winograd"),
                                                  ("phi_optimal", "phi_optimal"), ("cubic8", "cubic")])
def test_library_tables_equal_the_exact_tables_bitwise_in_fp32(lib_name, oracle_name):
    got = P.get(lib_name)
    want = [np.array(R.to_float(X), dtype=np.float64).astype(np.float32) for X in R.NAMED[oracle_name]()]
    for g, w, which in zip(got, want, "UVW"):
        assert g.dtype == np.float32 and g.shape == w.shape
        assert np.array_equal(g.view(np.uint32), w.view(np.uint32)), f"{lib_name}: {which} differs"


def test_library_phi_matches_exact_phi():
    for lib_name, oracle_name in (("strassen", "strassen"), ("winograd", "winograd"), ("phi_optimal", "phi_optimal")):
        assert P.phi(*P.get64(lib_name)) == pytest.approx(float(R.phi(*R.NAMED[oracle_name]())), rel=1e-14)
