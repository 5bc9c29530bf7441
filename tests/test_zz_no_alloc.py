"""GPU check of fmm_error_stats_noalloc, the entry point for callers that must not allocate device
memory (fixed-pool services, plugins, code that cannot afford cudaMalloc's implicit synchronisation).
It has to agree with fmm_error_stats, which takes caller-owned scratch, on two calls in a row: the
second call runs on top of whatever the first one left in the library's built-in scratch array.
Collected last on purpose, so a run that stops at the first failure has already run everything else."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_26077_b200 import fmm

pytestmark = pytest.mark.gpu


def _stats_pair(rows, cols, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    Cm = torch.randn(rows, cols, device="cuda", generator=g)
    Cref = Cm.double() + 1e-2 * torch.randn(rows, cols, device="cuda", generator=g, dtype=torch.float64)
    want = fmm.fmm_error_stats(Cm, Cref).cpu().numpy()
    out3 = torch.full((3,), float("nan"), dtype=torch.float64, device="cuda")
    got = fmm.fmm_error_stats_noalloc(Cm, Cref, out3).cpu().numpy()
    # ... and both against the CPU oracle's definition of the three statistics
    truth = O.error_stats(Cm.cpu().numpy().astype(np.float64), Cref.cpu().numpy())
    assert got[0] == pytest.approx(truth[0], rel=1e-12) and got[1] == pytest.approx(truth[1], rel=1e-12)
    assert got[2] == truth[2]
    return got, want


def test_noalloc_matches_scratch_version_twice_in_a_row():
    # two different problems back to back: the second must not see anything of the first
    for rows, cols, seed in ((1024, 768, 1), (384, 250, 2)):
        got, want = _stats_pair(rows, cols, seed)
        # same kernels, same block partition, same reduction order: the results are identical
        assert np.array_equal(got, want), (got, want)
        assert got[0] > 0 and got[1] > 0 and got[2] > 0
    torch.cuda.synchronize()


def test_noalloc_two_calls_queued_on_one_side_stream():
    # Callers may queue calls on their own stream without synchronising in between: the stream orders the two
    # calls' use of the shared array.  Different inputs per call, one synchronise at the end.
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    probs = []
    for rows, cols in ((512, 640), (256, 130)):
        Cm = torch.randn(rows, cols, device="cuda", generator=g)
        Cref = Cm.double() + 1e-3 * torch.randn(rows, cols, device="cuda", generator=g, dtype=torch.float64)
        probs.append((Cm, Cref, torch.full((3,), float("nan"), dtype=torch.float64, device="cuda")))
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    lib = fmm.lib()
    p = lambda t: C.c_void_p(t.data_ptr())
    with torch.cuda.stream(side):
        for Cm, Cref, out3 in probs:
            rc = lib.fmm_error_stats_noalloc(p(Cm), p(Cref), C.c_int64(Cm.shape[0]), C.c_int64(Cm.shape[1]), p(out3),
                                             C.c_void_p(side.cuda_stream))
            assert rc == 0
    side.synchronize()
    for Cm, Cref, out3 in probs:
        want = fmm.fmm_error_stats(Cm, Cref).cpu().numpy()
        assert np.array_equal(out3.cpu().numpy(), want)
        truth = O.error_stats(Cm.cpu().numpy().astype(np.float64), Cref.cpu().numpy())
        assert want[0] == pytest.approx(truth[0], rel=1e-12) and want[2] == truth[2]
    torch.cuda.synchronize()


def test_noalloc_rejects_oversize_and_bad_arguments():
    lib = fmm.lib()
    limit = lib.fmm_error_stats_noalloc_max_elements()
    assert limit == 1 << 28
    x = torch.zeros(4, device="cuda")
    r = torch.zeros(4, device="cuda", dtype=torch.float64)
    o = torch.zeros(3, device="cuda", dtype=torch.float64)
    p = lambda t: C.c_void_p(t.data_ptr())
    # one element beyond the limit (nothing is launched, so the small buffers are never touched)
    assert lib.fmm_error_stats_noalloc(p(x), p(r), C.c_int64(limit // 2 + 1), C.c_int64(2), p(o), None) == 2
    assert lib.fmm_error_stats_noalloc(p(x), p(r), C.c_int64(3), C.c_int64(3), p(o), None) == 2      # odd count
    # huge dimensions are refused before their product is formed
    assert lib.fmm_error_stats_noalloc(p(x), p(r), C.c_int64(1 << 62), C.c_int64(4), p(o), None) == 2
    assert lib.fmm_error_stats_noalloc(p(x), p(r), C.c_int64(1 << 40), C.c_int64(1 << 40), p(o), None) == 2
    assert lib.fmm_error_stats_noalloc(None, p(r), C.c_int64(2), C.c_int64(2), p(o), None) == 1
    assert lib.fmm_error_stats_noalloc(p(x), p(r), C.c_int64(2), C.c_int64(2), p(o), None) == 0
    torch.cuda.synchronize()
