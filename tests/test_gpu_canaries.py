"""Stand-in for a memory checker, part 1: canary margins.

Every buffer a call writes (workspace, C) sits inside a larger allocation whose margins hold a pattern; after
fmm_matmul at 0..3 recursion levels in every mode the margins must be untouched, the inputs unchanged, and the result
identical to the one computed with ordinary buffers."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2609_26077_b200 import fmm, workloads as Wl
from gpu_common import dev, make_plan

pytestmark = pytest.mark.gpu

MARGIN = 4096
PATTERN = 0xA5


def _guarded(nbytes, align):
    """A uint8 device buffer of nbytes with MARGIN bytes of pattern on both sides; the interior is `align`-aligned."""
    raw = torch.full((nbytes + 2 * MARGIN + align,), PATTERN, dtype=torch.uint8, device="cuda")
    off = MARGIN + (-(raw.data_ptr() + MARGIN)) % align
    return raw, off


def _margins_intact(raw, off, nbytes):
    return bool((raw[:off] == PATTERN).all()) and bool((raw[off + nbytes:] == PATTERN).all())


CASES = [(mode, blk, lv) for mode, blk in (("fp32", 32), ("fp32", 128), ("ue8m0", 32)) for lv in (0, 1, 2, 3)]


@pytest.mark.parametrize("mode,blk,levels", CASES)
def test_nothing_is_written_outside_workspace_and_output(mode, blk, levels):
    d = 1 << levels
    M, K, N = 256 * d, 128 * d, 384 * d          # rectangular, several tiles, single and paired CTAs
    if levels == 3:
        M, K, N = 128 * d, 128 * d, 128 * d
    A, B = Wl.gaussian(M, K, N, seed=11 + levels)
    a, b = dev(A), dev(B)
    plan = make_plan("winograd" if levels else "cubic", levels, blk, mode)
    want = plan.matmul(a, b, workspace=plan.workspace(M, N, K)).clone()
    ws_bytes = plan.workspace_bytes(M, N, K)
    ws_raw, ws_off = _guarded(ws_bytes, 1024)
    c_raw, c_off = _guarded(M * N * 4, 16)
    a0, b0 = a.clone(), b.clone()
    rc = fmm.lib().fmm_matmul(plan._h, C.c_void_p(a.data_ptr()), C.c_void_p(b.data_ptr()),
                              C.c_void_p(c_raw.data_ptr() + c_off), C.c_int64(M), C.c_int64(N), C.c_int64(K),
                              C.c_void_p(ws_raw.data_ptr() + ws_off), C.c_size_t(ws_bytes), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    assert _margins_intact(ws_raw, ws_off, ws_bytes), "a kernel wrote outside the workspace"
    assert _margins_intact(c_raw, c_off, M * N * 4), "a kernel wrote outside C"
    assert torch.equal(a, a0) and torch.equal(b, b0), "an input was modified"
    got = c_raw[c_off:c_off + M * N * 4].view(torch.float32).reshape(M, N)
    assert torch.equal(got, want)
    plan.close()


def test_statistics_and_reference_kernels_stay_inside_their_buffers():
    M, N, K = 192, 320, 64
    A, B = Wl.gaussian(M, K, N, seed=5)
    ref_raw, ref_off = _guarded(M * N * 8, 16)
    a, b = dev(A), dev(B)
    rc = fmm.lib().fmm_ref_gemm_fp64(C.c_void_p(a.data_ptr()), C.c_void_p(b.data_ptr()),
                                     C.c_void_p(ref_raw.data_ptr() + ref_off), C.c_int64(M), C.c_int64(N), C.c_int64(K), None)
    assert rc == 0
    scratch_bytes = fmm.lib().fmm_error_stats_scratch_bytes()
    sc_raw, sc_off = _guarded(scratch_bytes, 16)
    out_raw, out_off = _guarded(24, 16)
    Cm = torch.randn(M, N, device="cuda")
    rc = fmm.lib().fmm_error_stats(C.c_void_p(Cm.data_ptr()), C.c_void_p(ref_raw.data_ptr() + ref_off), C.c_int64(M),
                                   C.c_int64(N), C.c_void_p(out_raw.data_ptr() + out_off),
                                   C.c_void_p(sc_raw.data_ptr() + sc_off), C.c_size_t(scratch_bytes), None)
    assert rc == 0
    torch.cuda.synchronize()
    assert _margins_intact(ref_raw, ref_off, M * N * 8) and _margins_intact(sc_raw, sc_off, scratch_bytes)
    assert _margins_intact(out_raw, out_off, 24)
    ref = ref_raw[ref_off:ref_off + M * N * 8].view(torch.float64).reshape(M, N)
    assert torch.allclose(ref, a.double() @ b.double(), rtol=1e-12, atol=1e-12)
