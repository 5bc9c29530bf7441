"""GPU parity, whole path: C from fmm_matmul against the oracle's fp64 C on the same inputs.
Bar: relative Frobenius difference <= 1e-5 (accumulation-order differences only)."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_26077_b200 import fmm, workloads as Wl
from gpu_common import MODES, coeffs, dev, make_plan

pytestmark = pytest.mark.gpu
TOL = 1e-5

CASES = [
    ("cubic", 0, (128, 128, 128), 32, "ue8m0", "gaussian"),
    ("cubic", 0, (128, 128, 128), 32, "fp32", "gaussian"),
    ("cubic", 0, (256, 384, 512), 32, "ue8m0", "gaussian"),
    ("cubic", 0, (256, 384, 512), 32, "fp32", "gaussian"),
    ("cubic", 0, (384, 512, 256), 128, "fp32", "uniform"),
    ("strassen", 1, (256, 256, 256), 32, "fp32", "gaussian"),
    ("strassen", 1, (256, 256, 256), 32, "ue8m0", "gaussian"),
    ("phi_optimal", 1, (256, 768, 512), 32, "fp32", "gaussian"),
    ("phi_optimal", 1, (512, 256, 1024), 32, "ue8m0", "uniform"),
    ("winograd", 1, (512, 512, 512), 128, "fp32", "uniform"),
    ("cubic8", 1, (256, 256, 512), 32, "ue8m0", "gaussian"),
    ("phi_optimal", 2, (512, 512, 512), 32, "ue8m0", "llm"),
    ("strassen", 2, (512, 1024, 1024), 32, "fp32", "gaussian"),
    ("winograd", 3, (1024, 1024, 1024), 32, "ue8m0", "student_t3"),
    ("phi_optimal", 3, (1024, 1024, 1024), 32, "fp32", "scaled_gaussian"),
    ("phi_optimal", 1, (1024, 1024, 1024), 32, "ue8m0", "gaussian"),
    ("phi_optimal", 1, (1024, 1024, 1024), 32, "fp32", "gaussian"),
    ("phi_optimal", 1, (1024, 1024, 1024), 128, "fp32", "gaussian"),
    # orbit-panel arms: dense irrational coefficient tables (no compile-time zero pattern applies)
    ("pert_f1_shear_m_rb", 1, (512, 512, 512), 32, "fp32", "gaussian"),
    ("pert_f2_diag_p_rb", 1, (512, 512, 512), 32, "ue8m0", "uniform"),
    ("winograd_rb", 2, (512, 512, 512), 32, "ue8m0", "gaussian"),
    # more tile positions than CTA pairs / CTAs on a 148-SM part (80 positions on 74 pairs; 152 on 148 CTAs): several
    # work items per CTA (pair), spread evenly over the waves
    ("strassen", 1, (5120, 512, 4096), 32, "ue8m0", "gaussian"),
    ("phi_optimal", 1, (4864, 256, 4096), 32, "ue8m0", "uniform"),
    ("strassen", 1, (5120, 512, 4096), 128, "fp32", "gaussian"),
    # 16 or more K stages per term: fp32 / block-32 products take the kernel variant with the output warp
    ("cubic", 0, (256, 3072, 384), 32, "fp32", "gaussian"),
    ("phi_optimal", 1, (512, 6144, 768), 32, "fp32", "llm"),
    ("winograd", 1, (768, 8192, 256), 32, "fp32", "uniform"),
]


@pytest.mark.parametrize("name,levels,shape,blk,mode,family", CASES)
def test_matmul_matches_oracle(name, levels, shape, blk, mode, family):
    M, K, N = shape
    A, B = Wl.FAMILIES[family](M, K, N, seed=5)
    plan = make_plan(name, levels, blk, mode)
    C = plan.matmul(dev(A), dev(B))
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    U, V, W = coeffs(name)
    want = O.fused_fmm(A, B, U, V, W, levels=0 if name == "cubic" else levels, blk=blk, mode=MODES[mode])
    got = C.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert rel <= TOL, f"relative Frobenius difference {rel:.3e}"
    # every output block agrees, not just the whole (a misplaced block can hide in the norm)
    d = 1 << (0 if name == "cubic" else levels)
    for bi in range(d):
        for bj in range(d):
            sl = np.s_[bi * M // d:(bi + 1) * M // d, bj * N // d:(bj + 1) * N // d]
            r = np.linalg.norm(got[sl] - want[sl]) / np.linalg.norm(want[sl])
            assert r <= 2 * TOL, f"block ({bi},{bj}) differs by {r:.3e}"


def test_repeat_calls_are_bit_reproducible_and_overwrite_c():
    A, B = Wl.gaussian(512, 512, 512, 1)
    plan = make_plan("phi_optimal", 1, 32, "ue8m0")
    a, b = dev(A), dev(B)
    out = torch.full((512, 512), float("nan"), device="cuda")
    plan.matmul(a, b, out=out)
    c1 = out.clone()
    out.fill_(123.0)
    plan.matmul(a, b, out=out)
    torch.cuda.synchronize()
    assert torch.equal(c1, out)


def test_output_warp_variant_is_bit_reproducible():
    # 48 K stages per term: the fp32 / block-32 product runs the kernel variant whose post-addition is issued by a
    # dedicated warp while the next term is being promoted; the order of the add-reductions per tile is still fixed
    A, B = Wl.llm_shaped(512, 12288, 512, 2)
    plan = make_plan("phi_optimal", 1, 32, "fp32")
    a, b = dev(A), dev(B)
    c1 = plan.matmul(a, b).clone()
    for _ in range(3):
        assert torch.equal(plan.matmul(a, b), c1)
    assert plan.device_status() == (0, 0)


def test_errors_vs_fp64_reference_match_oracle_ratios():
    # the measured RMS error ratios between realizations must match the oracle's within 2 %
    n, seeds = 512, range(4)
    names = ["cubic", "strassen", "winograd", "phi_optimal"]
    for mode in ("fp32", "ue8m0"):
        g = {k: [] for k in names}
        o = {k: [] for k in names}
        for s in seeds:
            A, B = Wl.gaussian(n, n, n, s)
            a, b = dev(A), dev(B)
            ref_d = fmm.fmm_ref_gemm_fp64(a, b)
            ref_h = O.ref_gemm(A, B)
            for name in names:
                plan = make_plan(name, 1, 32, mode)
                g[name].append(fmm.rel_frobenius(plan.matmul(a, b), ref_d))
                U, V, W = coeffs(name)
                o[name].append(O.rel_frobenius(O.fused_fmm(A, B, U, V, W, levels=0 if name == "cubic" else 1,
                                                           blk=32, mode=MODES[mode]), ref_h))
        for name in names:
            ge, oe = np.mean(g[name]), np.mean(o[name])
            assert ge == pytest.approx(oe, rel=1e-3), (mode, name, ge, oe)
        for name in names[1:]:
            assert np.mean(g[name]) / np.mean(g["cubic"]) == pytest.approx(np.mean(o[name]) / np.mean(o["cubic"]), rel=0.02)
