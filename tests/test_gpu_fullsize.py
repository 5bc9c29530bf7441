"""GPU parity at the benchmark's full size (n = 8192, one level, Phi-optimal: the launch configuration
bench.py times).  The quantized operands are compared in full against the oracle; C is compared on
sampled rows and on sampled 128 x 128 tiles of every output block, which the oracle's own C code computes
entry by entry from its own quantized operands (plain loops, fp64)."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_26077_b200 import fmm, workloads as Wl
from gpu_common import MODES, coeffs, dev, make_plan

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode,blk,tile", [("fp32", 32, 0), ("ue8m0", 32, 0), ("fp32", 128, 0), ("fp32", 128, 128)])
def test_full_size_operands_bit_exact_and_sampled_rows_of_c(mode, blk, tile):
    # tile = 128: one weight-side scale per 128 x 128 tile (App. E.5), the fourth product-kernel mode bench.py times
    n = 8192
    h = n // 2
    A, B = Wl.gaussian(n, n, n, seed=0)
    plan = make_plan("phi_optimal", 1, blk, mode) if not tile else \
        fmm.Plan(*coeffs("phi_optimal"), levels=1, block_k=blk, scale_mode=mode, b_tile_n=tile)
    ws = plan.workspace(n, n, n)
    C = plan.matmul(dev(A), dev(B), workspace=ws)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    U, V, W = coeffs("phi_optimal")
    ca, sa, ea = O.encode(A, "A", U, V, 1, blk, MODES[mode])
    cb, sb, eb = O.encode(B, "B", U, V, 1, blk, MODES[mode], b_tile=tile)
    rng = np.random.default_rng(1)
    rows = np.sort(rng.choice(h, size=24, replace=False))
    # four 128 x 128 tiles of the leaf index space (each is compared in all four output blocks), not aligned to the
    # kernel's 256-row / 256-column tile positions
    tiles = [(int(r), int(c)) for r, c in zip(rng.integers(0, h - 128, 4), rng.integers(0, h - 128, 4))]
    allcols = np.arange(h)
    Mrows, Mtiles = [], []
    for t in range(7):
        qa, sca = plan.quantized_operand(ws, n, n, n, t, "A")
        qb, scb = plan.quantized_operand(ws, n, n, n, t, "B")
        assert np.array_equal(qa, ca[t]) and np.array_equal(qb, cb[t]), f"codes differ in term {t}"
        assert np.array_equal(sca, sa[t] if mode == "fp32" else ea[t]), f"A scales differ in term {t}"
        assert np.array_equal(scb, sb[t] if mode == "fp32" else eb[t]), f"B scales differ in term {t}"
        Mrows.append(O.leaf_product_sample(ca[t], sa[t], cb[t], sb[t], blk, rows, allcols))
        Mtiles.append([O.leaf_product_sample(ca[t], sa[t], cb[t], sb[t], blk, np.arange(r, r + 128), np.arange(c, c + 128))
                       for r, c in tiles])
    got = C.cpu().numpy().astype(np.float64)
    for q in range(4):
        r0, c0 = (q >> 1) * h, (q & 1) * h
        want = sum(float(W[r][q]) * Mrows[r] for r in range(7))
        block = got[r0 + rows][:, c0:c0 + h]
        rel = np.linalg.norm(block - want) / np.linalg.norm(want)
        assert rel <= 1e-5, f"quadrant {q}: sampled rows differ by {rel:.3e}"
        for i, (tr, tc) in enumerate(tiles):
            want = sum(float(W[r][q]) * Mtiles[r][i] for r in range(7))
            tile = got[r0 + tr:r0 + tr + 128, c0 + tc:c0 + tc + 128]
            rel = np.linalg.norm(tile - want) / np.linalg.norm(want)
            assert rel <= 1e-5, f"quadrant {q}, tile at ({tr},{tc}): differs by {rel:.3e}"
    assert np.isfinite(got).all()


def test_full_size_two_levels_operands_bit_exact_and_sampled_rows_of_c():
    # n = 8192 at two recursion levels (49 leaf products of 2048^3; fused two-level encoders, term groups as work
    # items, outer decoder as a separate kernel): all leaf operands in full, C on sampled leaf rows of all 16 blocks
    n, blk, mode = 8192, 32, "ue8m0"
    leaf = n // 4
    A, B = Wl.gaussian(n, n, n, seed=0)
    plan = make_plan("phi_optimal", 2, blk, mode)
    ws = plan.workspace(n, n, n)
    C = plan.matmul(dev(A), dev(B), workspace=ws)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    U, V, W = coeffs("phi_optimal")
    ca, sa, ea = O.encode(A, "A", U, V, 2, blk, MODES[mode])
    cb, sb, eb = O.encode(B, "B", U, V, 2, blk, MODES[mode])
    assert len(ca) == 49
    rng = np.random.default_rng(2)
    rows = np.sort(rng.choice(leaf, size=12, replace=False))
    Mrows = []
    for t in range(49):                                  # t = 7 * (outer term) + (inner term)
        qa, sca = plan.quantized_operand(ws, n, n, n, t, "A")
        qb, scb = plan.quantized_operand(ws, n, n, n, t, "B")
        assert np.array_equal(qa, ca[t]) and np.array_equal(qb, cb[t]), f"codes differ in term {t}"
        assert np.array_equal(sca, ea[t]) and np.array_equal(scb, eb[t]), f"scales differ in term {t}"
        Mrows.append(O.leaf_product_sample(ca[t], sa[t], cb[t], sb[t], blk, rows, np.arange(leaf)))
    got = C.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    for q1 in range(4):
        for q2 in range(4):
            want = sum(float(W[t1][q1]) * float(W[t2][q2]) * Mrows[7 * t1 + t2] for t1 in range(7) for t2 in range(7)
                       if W[t1][q1] != 0 and W[t2][q2] != 0)
            r0 = (q1 >> 1) * 2 * leaf + (q2 >> 1) * leaf
            c0 = (q1 & 1) * 2 * leaf + (q2 & 1) * leaf
            block = got[r0 + rows][:, c0:c0 + leaf]
            rel = np.linalg.norm(block - want) / np.linalg.norm(want)
            assert rel <= 1e-5, f"block ({q1},{q2}): sampled rows differ by {rel:.3e}"


def test_full_size_rectangular_llm_shape_sampled_rows_of_c():
    # M, K, N = 16384, 8192, 8192 with per-column outlier channels in A and small-variance weights in B: the quantized
    # operands in full, C on sampled rows of each output block
    M, K, N, blk, mode = 16384, 8192, 8192, 32, "fp32"
    A, B = Wl.FAMILIES["llm"](M, K, N, seed=3)
    plan = make_plan("strassen", 1, blk, mode)
    ws = plan.workspace(M, N, K)
    C = plan.matmul(dev(A), dev(B), workspace=ws)
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    U, V, W = coeffs("strassen")
    ca, sa, _ = O.encode(A, "A", U, V, 1, blk, MODES[mode])
    cb, sb, _ = O.encode(B, "B", U, V, 1, blk, MODES[mode])
    rng = np.random.default_rng(4)
    rows = np.sort(rng.choice(M // 2, size=16, replace=False))
    Mrows = []
    for t in range(7):
        qa, sca = plan.quantized_operand(ws, M, N, K, t, "A")
        qb, scb = plan.quantized_operand(ws, M, N, K, t, "B")
        assert np.array_equal(qa, ca[t]) and np.array_equal(qb, cb[t]), f"codes differ in term {t}"
        assert np.array_equal(sca, sa[t]) and np.array_equal(scb, sb[t]), f"scales differ in term {t}"
        Mrows.append(O.leaf_product_sample(ca[t], sa[t], cb[t], sb[t], blk, rows, np.arange(N // 2)))
    got = C.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    for q in range(4):
        want = sum(float(W[r][q]) * Mrows[r] for r in range(7) if W[r][q] != 0)
        r0, c0 = (q >> 1) * (M // 2), (q & 1) * (N // 2)
        block = got[r0 + rows][:, c0:c0 + N // 2]
        rel = np.linalg.norm(block - want) / np.linalg.norm(want)
        assert rel <= 1e-5, f"quadrant {q}: sampled rows differ by {rel:.3e}"
