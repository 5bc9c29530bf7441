"""GPU parity for the deployment-matched weight-side options (App. E.5): one FP32 scale per 128 x 128 tile of
each encoded B-side combination, optional bf16 pre-round.  Codes and scales bit-exact, C within 1e-5."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_26077_b200 import fmm, realizations as P, workloads as Wl
from gpu_common import coeffs, dev

pytestmark = pytest.mark.gpu

CASES = [
    ("cubic", 0, (128, 256, 384), "gaussian", False),      # unsplit B (N not a multiple of 512)
    ("cubic", 0, (256, 256, 1024), "llm", True),           # four column panels
    ("strassen", 1, (256, 512, 512), "gaussian", False),
    ("phi_optimal", 1, (512, 512, 768), "llm", True),
    ("winograd", 2, (512, 1024, 1024), "student_t3", True),
    ("pert_f0_diag_p_rb", 1, (256, 256, 512), "uniform", True),
    # 80 tile positions on 74 CTA pairs: two waves of 40 pairs
    ("strassen", 1, (5120, 512, 4096), "llm", False),
]


@pytest.mark.parametrize("name,levels,shape,family,bf16", CASES)
def test_tile_scales_match_oracle(name, levels, shape, family, bf16):
    M, K, N = shape
    A, B = Wl.FAMILIES[family](M, K, N, seed=11)
    U, V, W = coeffs(name)
    lv = 0 if name == "cubic" else levels
    plan = fmm.Plan(U, V, W, levels=lv, block_k=128, scale_mode="fp32", b_tile_n=128, b_preround_bf16=bf16)
    a, b = dev(A), dev(B)
    ws = plan.workspace(M, N, K)
    plan.encode_only(a, b, workspace=ws)
    torch.cuda.synchronize()
    want_c, want_s, _ = O.encode(B, "B", U, V, lv, blk=128, b_tile=128, b_bf16=bf16)
    for t in range(want_c.shape[0]):
        codes, scales = plan.quantized_operand(ws, M, N, K, t, "B")
        assert np.array_equal(codes, want_c[t]), f"codes of term {t}"
        assert np.array_equal(scales.view(np.uint32), want_s[t].view(np.uint32)), f"scales of term {t}"
    # the A side is untouched by the options
    a_c, a_s, _ = O.encode(A, "A", U, V, lv, blk=128)
    codes, scales = plan.quantized_operand(ws, M, N, K, 0, "A")
    assert np.array_equal(codes, a_c[0]) and np.array_equal(scales, a_s[0])
    C = plan.matmul(a, b, workspace=ws)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    want = O.fused_fmm(A, B, U, V, W, levels=lv, blk=128, b_tile=128, b_bf16=bf16)
    got = C.cpu().numpy().astype(np.float64)
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert rel <= 1e-5, f"relative Frobenius difference {rel:.3e}"


def test_bf16_preround_alone_matches_oracle():
    M, K, N = 256, 512, 512
    A, B = Wl.gaussian(M, K, N, 3)
    U, V, W = P.get("phi_optimal")
    plan = fmm.Plan(U, V, W, levels=1, block_k=128, scale_mode="fp32", b_preround_bf16=True)
    ws = plan.workspace(M, N, K)
    plan.encode_only(dev(A), dev(B), workspace=ws)
    torch.cuda.synchronize()
    want_c, want_s, _ = O.encode(B, "B", U, V, 1, blk=128, b_bf16=True)
    plain_c, _, _ = O.encode(B, "B", U, V, 1, blk=128)
    assert not np.array_equal(want_c, plain_c)          # the option does change the bytes
    for t in range(7):
        codes, scales = plan.quantized_operand(ws, M, N, K, t, "B")
        assert np.array_equal(codes, want_c[t])
        assert np.array_equal(scales.view(np.uint32), want_s[t].view(np.uint32))


def test_options_are_validated():
    U, V, W = P.get("strassen")
    for kw in (dict(block_k=32, scale_mode="fp32"), dict(block_k=32, scale_mode="ue8m0")):
        with pytest.raises(fmm.FmmError):
            fmm.Plan(U, V, W, levels=1, b_tile_n=128, **kw)
    with pytest.raises(fmm.FmmError):
        fmm.Plan(U, V, W, levels=1, block_k=128, b_tile_n=64)
