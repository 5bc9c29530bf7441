"""GPU parity, steps 1-2: the quantized leaf operands (e4m3 bytes and scales) produced by the
pre-addition + quantization kernels must be bit-identical to the oracle's."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_26077_b200 import workloads as Wl
from gpu_common import MODES, coeffs, dev, make_plan, oracle_scales

pytestmark = pytest.mark.gpu

CASES = [
    # name, levels, (M, K, N), blk, mode, family
    ("strassen", 1, (256, 256, 256), 32, "fp32", "gaussian"),
    ("phi_optimal", 1, (256, 768, 512), 32, "fp32", "gaussian"),
    ("winograd", 1, (512, 512, 256), 128, "fp32", "uniform"),
    ("phi_optimal", 1, (512, 256, 512), 32, "ue8m0", "gaussian"),
    ("cubic", 0, (256, 384, 128), 32, "fp32", "gaussian"),
    ("cubic", 0, (128, 256, 256), 32, "ue8m0", "student_t3"),
    ("cubic", 0, (128, 256, 128), 128, "fp32", "scaled_gaussian"),
    ("strassen", 2, (512, 512, 512), 32, "fp32", "gaussian"),
    ("phi_optimal", 2, (512, 1024, 512), 32, "ue8m0", "llm"),
    ("winograd", 3, (1024, 1024, 1024), 32, "fp32", "student_t3"),
    ("cubic8", 1, (256, 256, 256), 32, "fp32", "gaussian"),
    ("phi_optimal", 1, (256, 256, 256), 32, "fp32", "scaled_gaussian"),
    ("strassen", 1, (256, 256, 256), 128, "fp32", "student_t3"),
    # last two recursion levels in one kernel: rectangular shapes, every scale mode, a realization without a
    # pre-instantiated zero pattern, block 128 (two-level kernel on the A side only), three levels
    ("phi_optimal", 2, (512, 1536, 1024), 32, "fp32", "llm"),
    ("winograd", 2, (1024, 512, 1536), 32, "ue8m0", "student_t3"),
    ("pert_f1_diag_m_rb", 2, (512, 512, 1024), 32, "ue8m0", "gaussian"),
    ("pert_f2_shear_p_rb", 2, (512, 1024, 512), 32, "fp32", "uniform"),
    ("phi_optimal", 2, (512, 1024, 512), 128, "fp32", "gaussian"),
    ("cubic8", 2, (512, 512, 512), 32, "ue8m0", "gaussian"),
    ("phi_optimal", 3, (1024, 1024, 2048), 32, "ue8m0", "scaled_gaussian"),
]


@pytest.mark.parametrize("name,levels,shape,blk,mode,family", CASES)
def test_quantized_operands_bit_exact(name, levels, shape, blk, mode, family):
    M, K, N = shape
    A, B = Wl.FAMILIES[family](M, K, N, seed=11)
    plan = make_plan(name, levels, blk, mode)
    ws = plan.encode_only(dev(A), dev(B))
    torch.cuda.synchronize()
    U, V, _ = coeffs(name)
    ca, sa, ea = O.encode(A, "A", U, V, levels, blk, MODES[mode])
    cb, sb, eb = O.encode(B, "B", U, V, levels, blk, MODES[mode])
    wa, wb = oracle_scales(sa, ea, mode), oracle_scales(sb, eb, mode)
    for t in range(plan.terms):
        qa, sca = plan.quantized_operand(ws, M, N, K, t, "A")
        qb, scb = plan.quantized_operand(ws, M, N, K, t, "B")
        assert np.array_equal(qa, ca[t]), f"A codes differ in term {t}: {(qa != ca[t]).sum()} bytes"
        assert np.array_equal(qb, cb[t]), f"B codes differ in term {t}: {(qb != cb[t]).sum()} bytes"
        assert np.array_equal(sca.view(np.uint32) if mode == "fp32" else sca,
                              wa[t].view(np.uint32) if mode == "fp32" else wa[t]), f"A scales differ in term {t}"
        assert np.array_equal(scb.view(np.uint32) if mode == "fp32" else scb,
                              wb[t].view(np.uint32) if mode == "fp32" else wb[t]), f"B scales differ in term {t}"
    assert plan.device_status() == (0, 0)


def test_degenerate_blocks_zero_tiny_huge():
    # all-zero blocks (clamped scale), blocks below the 1e-12 clamp, huge magnitudes, signed zeros
    M = K = N = 256
    A, B = Wl.gaussian(M, K, N, 3)
    A[:64, :64] = 0.0
    A[64:128, :] *= np.float32(1e-14)
    A[128:192, 32:64] *= np.float32(1e30)
    A[200, :32] = -0.0
    B[:, :32] = 0.0
    B[:32, 64:128] *= np.float32(3e-13)
    B[96:128, :] *= np.float32(1e25)
    for mode in ("fp32", "ue8m0"):
        plan = make_plan("phi_optimal", 1, 32, mode)
        ws = plan.encode_only(dev(A), dev(B))
        U, V, _ = coeffs("phi_optimal")
        ca, sa, ea = O.encode(A, "A", U, V, 1, 32, MODES[mode])
        cb, sb, eb = O.encode(B, "B", U, V, 1, 32, MODES[mode])
        for t in range(7):
            qa, sca = plan.quantized_operand(ws, M, N, K, t, "A")
            qb, scb = plan.quantized_operand(ws, M, N, K, t, "B")
            assert np.array_equal(qa, ca[t]) and np.array_equal(qb, cb[t])
            assert np.array_equal(sca, oracle_scales(sa, ea, mode)[t])
            assert np.array_equal(scb, oracle_scales(sb, eb, mode)[t])


def test_hardware_cast_matches_oracle_on_every_rounding_boundary():
    # one block whose amax is exactly 448 gives scale 1 and inv 1: the stored codes are then the
    # device's e4m3 cast of the inputs themselves; feed every midpoint and its fp32 neighbours
    d = O.e4m3_decode(np.arange(0x7F, dtype=np.uint8))
    mids = ((d[:-1] + d[1:]) / 2).astype(np.float32)
    vals = np.concatenate([mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(np.inf)),
                           d.astype(np.float32), np.float32([1e-8, 2.0 ** -10, 2.0 ** -11])])
    vals = np.concatenate([vals, -vals])
    n = 32 * ((vals.size + 30) // 31)
    x = np.zeros(n, np.float32)
    blocks = x.reshape(-1, 32)
    blocks[:, 0] = 448.0
    blocks[:, 1:].reshape(-1)[:vals.size] = vals
    K = ((max(256, n) + 127) // 128) * 128
    A = np.zeros((128, K), np.float32)
    A[0, :n] = x
    B = np.zeros((K, 128), np.float32)
    plan = make_plan("cubic", 0, 32, "fp32")
    ws = plan.encode_only(dev(A), dev(B))
    qa, sca = plan.quantized_operand(ws, 128, 128, K, 0, "A")
    ca, sa, _ = O.quant_rows(A, 32)
    assert np.array_equal(sca, sa) and sa[0, 0] == 1.0
    assert np.array_equal(qa, ca)
    assert np.array_equal(qa[0, :n], O.e4m3_encode(x))
