"""GPU parity over seeded random shapes: every kernel variant the dispatcher can pick (single CTA / CTA pair,
128- / 256-column tiles, every scale mode, weight tiles, one to three levels) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_26077_b200 import fmm, workloads as Wl
from gpu_common import MODES, coeffs, dev

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.default_rng(20260926)
    names = ["cubic", "strassen", "winograd", "phi_optimal", "pert_f0_shear_m_rb"]
    quant = [(32, "fp32", 0), (32, "ue8m0", 0), (128, "fp32", 0), (128, "fp32", 128)]
    out = []
    for i in range(24):
        name = names[i % len(names)]
        lv = 0 if name == "cubic" else int(rng.integers(1, 4))
        unit = 128 << lv
        cap = 1536 if lv < 3 else 2048
        dims = [unit * int(rng.integers(1, max(2, cap // unit + 1))) for _ in range(3)]
        blk, mode, tile = quant[i % len(quant)]
        out.append((name, lv, tuple(dims), blk, mode, tile, 100 + i))
    return out


@pytest.mark.parametrize("name,levels,shape,blk,mode,tile,seed", _cases())
def test_random_shape_matches_oracle(name, levels, shape, blk, mode, tile, seed):
    M, K, N = shape
    fam = ["gaussian", "uniform", "llm", "student_t3"][seed % 4]
    A, B = Wl.FAMILIES[fam](M, K, N, seed)
    U, V, W = coeffs(name)
    plan = fmm.Plan(U, V, W, levels=levels, block_k=blk, scale_mode=mode, b_tile_n=tile)
    C = plan.matmul(dev(A), dev(B))
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    want = O.fused_fmm(A, B, U, V, W, levels=levels, blk=blk, mode=MODES[mode], b_tile=tile)
    got = C.cpu().numpy().astype(np.float64)
    rel = np.linalg.norm(got - want) / np.linalg.norm(want)
    assert np.isfinite(got).all() and rel <= 1e-5, f"{shape}: relative Frobenius difference {rel:.3e}"
