"""Stand-in for a memory checker, part 2: the range-checked build.

libfmm_b200_debug.so is the same source compiled with -DFMM_DEBUG: every global store of every kernel is tested
against the buffers its launch was given, a store outside them is skipped and a location code is recorded.  The whole
path runs under it here (child process, so that one interpreter never holds both builds): results still match the
oracle, no violation is recorded at any level or mode, and the guard's own self-test shows a violation is reported
without a fault."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import json, sys
import numpy as np, torch
sys.path.insert(0, %(root)r)
from paper_2609_26077_b200 import build, fmm, realizations as P, workloads as Wl
from oracle import oracle as O
build.build(debug=True)
assert fmm.lib().fmm_debug_build() == 1
import ctypes as C
def violation(plan):
    code = C.c_int(-1)
    assert fmm.lib().fmm_debug_violation(plan._h if plan is not None else None, C.byref(code)) == 0
    return code.value
out = {"cases": []}
for mode, omode, blk in (("fp32", O.SCALE_FP32, 32), ("fp32", O.SCALE_FP32, 128), ("ue8m0", O.SCALE_UE8M0, 32)):
    for levels in (0, 1, 2, 3):
        d = 1 << levels
        M, K, N = (256 * d, 128 * d, 384 * d) if levels < 3 else (128 * d, 128 * d, 128 * d)
        A, B = Wl.gaussian(M, K, N, seed=21 + levels)
        U, V, W = P.get("phi_optimal")
        plan = fmm.Plan(U, V, W, levels=levels, block_k=blk, scale_mode=mode) if levels else fmm.Plan(levels=0, block_k=blk, scale_mode=mode)
        a, b = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
        Cg = plan.matmul(a, b, workspace=plan.workspace(M, N, K))
        torch.cuda.synchronize()
        want = O.fused_fmm(A, B, U, V, W, levels=levels, blk=blk, mode=omode)
        got = Cg.cpu().numpy().astype(np.float64)
        rel = float(np.linalg.norm(got - want) / np.linalg.norm(want))
        fmm.fmm_ref_gemm_fp64(a[:, :64].contiguous(), b[:64].contiguous())      # reference kernel under its guard too
        out["cases"].append({"mode": mode, "blk": blk, "levels": levels, "rel": rel, "violation": violation(plan),
                             "status": plan.device_status()})
        plan.close()
# statistics kernels (no plan)
Cm = torch.randn(192, 320, device="cuda"); Cr = Cm.double() + 1e-3
stats = fmm.fmm_error_stats(Cm, Cr).cpu().numpy().tolist()
out["stats_violation"] = violation(None)
out["stats"] = stats
# the guard reports a bad store without a fault: self-test, then clear
plan = fmm.Plan(levels=0, block_k=32, scale_mode="fp32")
assert fmm.lib().fmm_selftest_store_guard(plan._h, None) == 0
out["selftest_violation"] = violation(plan)
plan.device_status_clear()
out["after_clear"] = violation(plan)
x = torch.randn(256, 256, device="cuda")
out["usable_after"] = bool(torch.isfinite(plan.matmul(x, x, workspace=plan.workspace(256, 256, 256))).all())
print("RESULT " + json.dumps(out))
"""


def test_whole_path_under_the_range_checked_build():
    env = dict(os.environ, FMM_B200_DEBUG="1")
    r = subprocess.run([sys.executable, "-c", CHILD % {"root": ROOT}], capture_output=True, text=True, timeout=900, env=env)
    assert r.returncode == 0, r.stderr[-3000:]
    line = [ln for ln in r.stdout.splitlines() if ln.startswith("RESULT ")][-1]
    out = json.loads(line[len("RESULT "):])
    assert len(out["cases"]) == 12
    for c in out["cases"]:
        assert c["violation"] == 0, c
        assert c["status"] == [0, 0], c
        assert c["rel"] <= 1e-5, c
    assert out["stats_violation"] == 0 and out["stats"][0] > 0
    assert out["selftest_violation"] == 1901          # reported, not trapped
    assert out["after_clear"] == 0 and out["usable_after"]
