"""GPU checks of the boundary's error behaviour, of properties that hold at any size, and of the
bounded-wait failure path (a wait that runs out must leave a status code and a usable context)."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2609_26077_b200 import fmm, realizations as P, workloads as Wl
from gpu_common import dev, make_plan

pytestmark = pytest.mark.gpu


def test_matmul_rejects_bad_shapes_workspace_and_pointers():
    plan = make_plan("strassen", 1, 32, "fp32")
    lib = fmm.lib()
    a = torch.zeros(256, 256, device="cuda")
    c = torch.zeros(256, 256, device="cuda")
    ws = plan.workspace(256, 256, 256)
    p = lambda t: C.c_void_p(t.data_ptr())
    call = lambda M, N, K, w, wb, A=a, B=a, Cc=c: lib.fmm_matmul(plan._h, p(A) if A is not None else None, p(B), p(Cc),
                                                                 C.c_int64(M), C.c_int64(N), C.c_int64(K), w, C.c_size_t(wb), None)
    assert call(256, 256, 256, p(ws), ws.numel()) == 0
    assert call(192, 256, 256, p(ws), ws.numel()) == 2          # M/2 not a multiple of 128
    assert call(256, 256, 320, p(ws), ws.numel()) == 2          # K/2 not a multiple of 128
    assert call(0, 256, 256, p(ws), ws.numel()) == 2
    assert call(256, 256, 256, p(ws), ws.numel() - 1) == 4      # workspace too small
    assert call(256, 256, 256, None, ws.numel()) == 4
    assert call(256, 256, 256, C.c_void_p(ws.data_ptr() + 8), ws.numel()) == 4   # misaligned
    assert call(256, 256, 256, p(ws), ws.numel(), A=None) == 1
    # operands that are not 16-byte aligned are refused before anything is launched (the kernels use vector loads)
    big = torch.zeros(256 * 256 + 4, device="cuda")
    odd = lambda off: C.c_void_p(big.data_ptr() + off)
    assert lib.fmm_matmul(plan._h, odd(4), p(a), p(c), C.c_int64(256), C.c_int64(256), C.c_int64(256), p(ws),
                          C.c_size_t(ws.numel()), None) == 1
    assert lib.fmm_matmul(plan._h, p(a), odd(8), p(c), C.c_int64(256), C.c_int64(256), C.c_int64(256), p(ws),
                          C.c_size_t(ws.numel()), None) == 1
    assert lib.fmm_matmul(plan._h, p(a), p(a), odd(4), C.c_int64(256), C.c_int64(256), C.c_int64(256), p(ws),
                          C.c_size_t(ws.numel()), None) == 1
    assert lib.fmm_matmul(plan._h, odd(16), p(a), p(c), C.c_int64(256), C.c_int64(256), C.c_int64(256), p(ws),
                          C.c_size_t(ws.numel()), None) == 0
    need = C.c_size_t()
    assert lib.fmm_workspace_bytes(plan._h, C.c_int64(100), C.c_int64(256), C.c_int64(256), C.byref(need)) == 2
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)


def test_power_of_two_rescaling_leaves_codes_identical_on_device():
    # App. E.2: Q(2^k x) has the same codes and 2^k-times the scales
    A, B = Wl.gaussian(256, 256, 256, 4)
    plan = make_plan("phi_optimal", 1, 32, "fp32")
    ws = plan.encode_only(dev(A), dev(B))
    q0, s0 = plan.quantized_operand(ws, 256, 256, 256, 4, "A")
    r0, t0 = plan.quantized_operand(ws, 256, 256, 256, 4, "B")
    ws = plan.encode_only(dev(A * np.float32(2.0 ** 9)), dev(B * np.float32(2.0 ** -13)))
    q1, s1 = plan.quantized_operand(ws, 256, 256, 256, 4, "A")
    r1, t1 = plan.quantized_operand(ws, 256, 256, 256, 4, "B")
    assert np.array_equal(q0, q1) and np.array_equal(r0, r1)
    assert np.array_equal(s1, s0 * np.float32(2.0 ** 9)) and np.array_equal(t1, t0 * np.float32(2.0 ** -13))


def test_term_permutation_and_cubic_realization_properties():
    # permuting the terms of a realization only changes the summation order of the decode;
    # the rank-8 cubic realization at one level quantizes the same blocks as the cubic product
    A, B = Wl.gaussian(512, 512, 512, 8)
    a, b = dev(A), dev(B)
    U, V, W = P.get("winograd")
    perm = np.array([3, 0, 6, 1, 5, 2, 4])
    c0 = fmm.Plan(U, V, W, levels=1, scale_mode="ue8m0").matmul(a, b).cpu().numpy().astype(np.float64)
    c1 = fmm.Plan(U[perm], V[perm], W[perm], levels=1, scale_mode="ue8m0").matmul(a, b).cpu().numpy().astype(np.float64)
    assert np.linalg.norm(c0 - c1) / np.linalg.norm(c0) < 1e-6
    c8 = fmm.Plan(*P.get("cubic8"), levels=1, scale_mode="fp32").matmul(a, b).cpu().numpy().astype(np.float64)
    cc = fmm.Plan(levels=0, scale_mode="fp32").matmul(a, b).cpu().numpy().astype(np.float64)
    assert np.linalg.norm(c8 - cc) / np.linalg.norm(cc) < 1e-6


def test_rademacher_operands_strassen_is_exact_up_to_scale_rounding():
    # Sec. 4.3: on +-1 operands Strassen's combinations are exactly representable after block scaling
    A, B = Wl.rademacher(256, 256, 256, 0)
    a, b = dev(A), dev(B)
    ref = fmm.fmm_ref_gemm_fp64(a, b)
    es = fmm.rel_frobenius(make_plan("strassen", 1, 32, "fp32").matmul(a, b), ref)
    ep = fmm.rel_frobenius(make_plan("phi_optimal", 1, 32, "fp32").matmul(a, b), ref)
    assert es < 1e-6 and ep > 1e-3
    es_mx = fmm.rel_frobenius(make_plan("strassen", 1, 32, "ue8m0").matmul(a, b), ref)
    assert es_mx == 0.0          # power-of-two scales: exact


def test_bounded_wait_runs_out_and_leaves_the_context_usable():
    plan = make_plan("strassen", 1, 32, "ue8m0")
    assert plan.device_status() == (0, 0)
    plan.selftest_bounded_wait(2_000_000)                 # 2 ms limit on a barrier nothing signals
    torch.cuda.synchronize()
    st, code = plan.device_status()
    assert st == 8 and code == 901                        # FMM_ERR_DEVICE_TIMEOUT, self-test location
    plan.device_status_clear()
    assert plan.device_status() == (0, 0)
    # the context still works: a real product after the timed-out wait matches the oracle
    A, B = Wl.gaussian(256, 256, 256, 2)
    got = plan.matmul(dev(A), dev(B)).cpu().numpy().astype(np.float64)
    want = O.fused_fmm(A, B, *P.get("strassen"), levels=1, blk=32, mode=O.SCALE_UE8M0)
    assert np.linalg.norm(got - want) / np.linalg.norm(want) < 1e-5
    assert plan.device_status() == (0, 0)


def test_matmul_can_be_captured_in_a_cuda_graph():
    # fmm_matmul allocates nothing and never synchronises with the host, so the whole path (encode, products,
    # decode; here two recursion levels = 5 launches) can be captured once and replayed
    M, K, N = 512, 512, 512
    A, B = Wl.gaussian(M, K, N, 21)
    a, b = dev(A), dev(B)
    for mode in ("fp32", "ue8m0"):
        plan = make_plan("phi_optimal", 2, 32, mode)
        ws = plan.workspace(M, N, K)
        eager = plan.matmul(a, b, workspace=ws).clone()          # also warms up (function attributes are set once)
        out = torch.zeros((M, N), device="cuda")
        stream = torch.cuda.Stream()
        stream.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            with torch.cuda.graph(graph, stream=stream):
                plan.matmul(a, b, out=out, workspace=ws, stream=stream)
        torch.cuda.current_stream().wait_stream(stream)
        for _ in range(3):
            out.fill_(float("nan"))
            graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, eager)
        assert plan.device_status() == (0, 0)


@pytest.mark.parametrize("pinned", [True, False])
def test_host_operand_call_matches_the_device_call_bit_for_bit(pinned):
    # fmm_matmul_host = upload, fmm_matmul, download: same kernels on the same bytes, so C is identical; two calls on two
    # streams with their own workspaces may overlap and must not disturb each other
    M, K, N = 512, 768, 256
    A, B = Wl.gaussian(M, K, N, 9)
    plan = make_plan("phi_optimal", 1, 32, "fp32")
    want = plan.matmul(dev(A), dev(B)).cpu()
    Ah, Bh = torch.from_numpy(A).clone(), torch.from_numpy(B).clone()
    if pinned:
        Ah, Bh = Ah.pin_memory(), Bh.pin_memory()
    streams = [torch.cuda.Stream() for _ in range(2)]
    wss = [plan.host_workspace(M, N, K) for _ in range(2)]
    outs = [torch.full((M, N), float("nan")) for _ in range(2)]
    if pinned:
        outs = [o.pin_memory() for o in outs]
    torch.cuda.synchronize()
    for rep in range(2):
        for i in range(2):
            plan.matmul_host(Ah, Bh, outs[i], wss[i], stream=streams[i])
    torch.cuda.synchronize()
    assert plan.device_status() == (0, 0)
    assert torch.equal(outs[0], want) and torch.equal(outs[1], want)


def test_host_operand_call_rejects_bad_arguments():
    plan = make_plan("strassen", 1, 32, "ue8m0")
    lib = fmm.lib()
    h = torch.zeros(256, 256)
    ws = plan.host_workspace(256, 256, 256)
    inner = plan.workspace_bytes(256, 256, 256)
    assert ws.numel() >= inner + 3 * 256 * 256 * 4
    p = lambda t: C.c_void_p(t.data_ptr())
    call = lambda M, w, wb, A=h: lib.fmm_matmul_host(plan._h, p(A) if A is not None else None, p(h), p(h), C.c_int64(M),
                                                     C.c_int64(256), C.c_int64(256), w, C.c_size_t(wb), None)
    assert call(256, p(ws), ws.numel()) == 0
    torch.cuda.synchronize()
    assert call(192, p(ws), ws.numel()) == 2
    assert call(256, p(ws), inner) == 4                 # room for the product's workspace only
    assert call(256, None, ws.numel()) == 4
    assert call(256, p(ws), ws.numel(), A=None) == 1
    need = C.c_size_t()
    assert lib.fmm_host_workspace_bytes(plan._h, C.c_int64(100), C.c_int64(256), C.c_int64(256), C.byref(need)) == 2
    assert lib.fmm_host_workspace_bytes(plan._h, C.c_int64(256), C.c_int64(256), C.c_int64(256), None) == 1
    assert lib.fmm_host_workspace_bytes(None, C.c_int64(256), C.c_int64(256), C.c_int64(256), C.byref(need)) == 1


def test_status_is_read_after_work_on_a_non_blocking_stream():
    # fmm_device_status waits for every stream of the device, also streams that do not synchronise with the
    # default stream (torch's side streams are of that kind): the timeout set by a kernel still running there is seen
    plan = make_plan("strassen", 1, 32, "ue8m0")
    side = torch.cuda.Stream()
    assert fmm.lib().fmm_selftest_bounded_wait(plan._h, C.c_int64(50_000_000), C.c_void_p(side.cuda_stream)) == 0
    assert plan.device_status() == (8, 901)             # read right away, no explicit synchronisation
    plan.device_status_clear()
    assert plan.device_status() == (0, 0)
    plan.close()


@pytest.mark.skipif(torch.cuda.device_count() < 2, reason="needs two devices")
def test_call_on_another_device_is_refused():
    plan = make_plan("strassen", 1, 32, "ue8m0")
    ws = plan.workspace(256, 256, 256)
    a = torch.zeros(256, 256, device="cuda:0")
    torch.cuda.set_device(1)
    try:
        rc = fmm.lib().fmm_matmul(plan._h, C.c_void_p(a.data_ptr()), C.c_void_p(a.data_ptr()), C.c_void_p(a.data_ptr()),
                                  C.c_int64(256), C.c_int64(256), C.c_int64(256), C.c_void_p(ws.data_ptr()),
                                  C.c_size_t(ws.numel()), None)
        assert rc == 9
    finally:
        torch.cuda.set_device(0)
    plan.close()


@pytest.mark.parametrize("mode,blk,levels", [("fp32", 32, 1), ("ue8m0", 32, 1), ("fp32", 128, 1), ("ue8m0", 32, 2), ("fp32", 32, 0)])
def test_work_enqueued_behind_a_call_sees_all_of_its_kernels_complete(mode, blk, levels):
    # The kernels of one call overlap each other (the B-side encoder starts under the A-side encoder's tail, the
    # product kernel is set up under the B side's); towards the rest of the stream the call must stay ordinary
    # stream-ordered work.  Device-to-device copies of the workspace and of C enqueued right behind a call, with no
    # synchronisation in between, must hold the finished bytes: they are compared with a second plan's synchronised run.
    M, K, N = 2048, 4096, 2048
    A, B = Wl.gaussian(M, K, N, seed=5)
    a, b = dev(A), dev(B)
    name = "phi_optimal" if levels else "cubic"
    plan, ref_plan = make_plan(name, levels, blk, mode), make_plan(name, levels, blk, mode)
    ws, ws_ref = plan.workspace(M, N, K), ref_plan.workspace(M, N, K)
    ws_ref.zero_()
    ref_plan.encode_only(a, b, workspace=ws_ref)
    torch.cuda.synchronize()
    want_encoded = ws_ref.clone()
    want_c = ref_plan.matmul(a, b, workspace=ws_ref)
    torch.cuda.synchronize()
    want_after = ws_ref.clone()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for rep in range(4):
            ws.zero_()
            plan.encode_only(a, b, workspace=ws, stream=s)
            snap_encoded = ws.clone()                         # enqueued behind the call on the same stream
            c = torch.full((M, N), float("nan"), device="cuda")
            plan.matmul(a, b, out=c, workspace=ws, stream=s)
            snap_c, snap_after = c.clone(), ws.clone()
    s.synchronize()
    assert plan.device_status() == (0, 0)
    assert torch.equal(snap_encoded, want_encoded), "workspace copied right behind fmm_encode_only"
    assert torch.equal(snap_after, want_after), "workspace copied right behind fmm_matmul"
    assert torch.equal(snap_c, want_c), "C copied right behind fmm_matmul"
