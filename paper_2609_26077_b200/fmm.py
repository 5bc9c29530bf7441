"""Thin ctypes binding of libfmm_b200.so (argument marshalling only; every step runs in the
CUDA kernels).  torch supplies device memory and streams.  Names follow include/fmm.h."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# FMM_B200_DEBUG=1 in the environment selects the checked build (-DFMM_DEBUG: every global store of every kernel is
# range-checked, see fmm_debug_violation); it is slower and meant for tests
LIB_PATH = os.path.join(_HERE, "libfmm_b200_debug.so" if os.environ.get("FMM_B200_DEBUG") == "1" else "libfmm_b200.so")

FMM_OK = 0
STATUS_NAMES = ["FMM_OK", "FMM_ERR_INVALID_ARG", "FMM_ERR_SHAPE", "FMM_ERR_NOT_EXACT", "FMM_ERR_WORKSPACE",
                "FMM_ERR_ALLOC", "FMM_ERR_CUDA", "FMM_ERR_ARCH", "FMM_ERR_DEVICE_TIMEOUT", "FMM_ERR_WRONG_DEVICE"]
SCALE_FP32, SCALE_UE8M0 = 0, 1
SCALE_MODES = {"fp32": SCALE_FP32, "ue8m0": SCALE_UE8M0}

EXPORTS = ["fmm_plan_create", "fmm_plan_destroy", "fmm_workspace_bytes", "fmm_matmul", "fmm_host_workspace_bytes",
           "fmm_matmul_host", "fmm_encode_only",
           "fmm_multiply_only", "fmm_quantized_view", "fmm_ref_gemm_fp64", "fmm_error_stats",
           "fmm_error_stats_scratch_bytes", "fmm_error_stats_noalloc", "fmm_error_stats_noalloc_max_elements",
           "fmm_device_status", "fmm_device_status_clear", "fmm_selftest_bounded_wait", "fmm_phi_gamma", "fmm_brent_residual",
           "fmm_last_launch_count", "fmm_status_string", "fmm_debug_build", "fmm_debug_violation",
           "fmm_selftest_store_guard"]


class QuantParams(C.Structure):
    _fields_ = [("block_k", C.c_int), ("scale_mode", C.c_int), ("amax_floor", C.c_float), ("fp8_max", C.c_float),
                ("b_tile_n", C.c_int), ("b_preround_bf16", C.c_int)]


class FmmError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{what}: {name} ({lib().fmm_status_string(status).decode()})")


_lib = None


def lib():
    """Load the CUDA library.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_26077_b200.build` "
                              "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.fmm_status_string.restype = C.c_char_p
        L.fmm_status_string.argtypes = [C.c_int]
        L.fmm_error_stats_scratch_bytes.restype = C.c_size_t
        L.fmm_error_stats_noalloc_max_elements.restype = C.c_int64
        L.fmm_debug_build.restype = C.c_int
        for name in EXPORTS:
            getattr(L, name)
        _lib = L
    return _lib


def _check(status, what):
    if status != FMM_OK:
        raise FmmError(status, what)


def _fptr(a):
    if a is None:
        return None
    return a.ctypes.data_as(C.POINTER(C.c_float))


def _coef(x):
    return None if x is None else np.ascontiguousarray(np.asarray(x, dtype=np.float32))


def fmm_phi_gamma(U, V, W):
    U, V, W = _coef(U), _coef(V), _coef(W)
    phi, gam = C.c_double(), C.c_double()
    _check(lib().fmm_phi_gamma(C.c_int(U.shape[0]), _fptr(U), _fptr(V), _fptr(W), C.byref(phi), C.byref(gam)),
           "fmm_phi_gamma")
    return phi.value, gam.value


def fmm_brent_residual(U, V, W):
    U, V, W = _coef(U), _coef(V), _coef(W)
    r = C.c_double()
    _check(lib().fmm_brent_residual(C.c_int(U.shape[0]), _fptr(U), _fptr(V), _fptr(W), C.byref(r)), "fmm_brent_residual")
    return r.value


def _stream_ptr(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _dev_ptr(t):
    return C.c_void_p(t.data_ptr())


class Plan:
    """fmm_plan_create / fmm_plan_destroy plus the calls that take a plan."""

    def __init__(self, U=None, V=None, W=None, levels=1, block_k=32, scale_mode="fp32", amax_floor=1e-12,
                 b_tile_n=0, b_preround_bf16=False):
        self.U, self.V, self.W = _coef(U), _coef(V), _coef(W)
        self.levels = int(levels)
        self.block_k = int(block_k)
        self.scale_mode = SCALE_MODES[scale_mode] if isinstance(scale_mode, str) else int(scale_mode)
        self.rank = 0 if self.U is None else int(self.U.shape[0])
        qp = QuantParams(self.block_k, self.scale_mode, float(amax_floor), 448.0, int(b_tile_n), int(bool(b_preround_bf16)))
        h = C.c_void_p()
        _check(lib().fmm_plan_create(C.byref(h), C.c_int(self.rank), _fptr(self.U), _fptr(self.V), _fptr(self.W),
                                     C.c_int(self.levels), C.byref(qp)), "fmm_plan_create")
        self._h = h
        self._ws = None

    def close(self):
        if getattr(self, "_h", None):
            lib().fmm_plan_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def terms(self):
        return (self.rank ** self.levels) if self.levels > 0 else 1

    def workspace_bytes(self, M, N, K):
        b = C.c_size_t()
        _check(lib().fmm_workspace_bytes(self._h, C.c_int64(M), C.c_int64(N), C.c_int64(K), C.byref(b)),
               "fmm_workspace_bytes")
        return b.value

    def workspace(self, M, N, K, device="cuda"):
        """A torch byte tensor large enough for this size (cached; 1024-byte aligned)."""
        import torch
        need = self.workspace_bytes(M, N, K)
        if self._ws is None or self._ws.numel() < need + 1024 or str(self._ws.device) != str(torch.device(device)):
            self._ws = torch.empty(need + 1024, dtype=torch.uint8, device=device)
        off = (-self._ws.data_ptr()) % 1024
        return self._ws[off:off + need]

    def matmul(self, A, B, out=None, workspace=None, stream=None):
        """fmm_matmul: C = A @ B through the realization, all steps on the device."""
        import torch
        M, K = A.shape
        K2, N = B.shape
        assert K == K2 and A.dtype == torch.float32 and B.dtype == torch.float32
        assert A.is_contiguous() and B.is_contiguous() and A.is_cuda and B.is_cuda
        if out is None:
            out = torch.empty((M, N), dtype=torch.float32, device=A.device)
        ws = workspace if workspace is not None else self.workspace(M, N, K, A.device)
        _check(lib().fmm_matmul(self._h, _dev_ptr(A), _dev_ptr(B), _dev_ptr(out), C.c_int64(M), C.c_int64(N),
                                C.c_int64(K), _dev_ptr(ws), C.c_size_t(ws.numel()), _stream_ptr(stream)), "fmm_matmul")
        return out

    def host_workspace(self, M, N, K, device="cuda"):
        """Device buffer for matmul_host: fmm_host_workspace_bytes, 1024-byte aligned (a fresh tensor per call)."""
        import torch
        need = C.c_size_t()
        _check(lib().fmm_host_workspace_bytes(self._h, C.c_int64(M), C.c_int64(N), C.c_int64(K), C.byref(need)),
               "fmm_host_workspace_bytes")
        buf = torch.empty(need.value + 1024, dtype=torch.uint8, device=device)
        off = (-buf.data_ptr()) % 1024
        return buf[off:off + need.value]

    def matmul_host(self, A, B, out, workspace, stream=None):
        """fmm_matmul_host: host operands (pinned for asynchronous copies), C written to the host tensor `out`."""
        import torch
        M, K = A.shape
        K2, N = B.shape
        assert K == K2 and tuple(out.shape) == (M, N)
        for t in (A, B, out):
            assert t.dtype == torch.float32 and t.is_contiguous() and not t.is_cuda
        _check(lib().fmm_matmul_host(self._h, C.c_void_p(A.data_ptr()), C.c_void_p(B.data_ptr()), C.c_void_p(out.data_ptr()),
                                     C.c_int64(M), C.c_int64(N), C.c_int64(K), _dev_ptr(workspace),
                                     C.c_size_t(workspace.numel()), _stream_ptr(stream)), "fmm_matmul_host")
        return out

    def encode_only(self, A, B, workspace=None, stream=None):
        M, K = A.shape
        _, N = B.shape
        ws = workspace if workspace is not None else self.workspace(M, N, K, A.device)
        _check(lib().fmm_encode_only(self._h, _dev_ptr(A), _dev_ptr(B), C.c_int64(M), C.c_int64(N), C.c_int64(K),
                                     _dev_ptr(ws), C.c_size_t(ws.numel()), _stream_ptr(stream)), "fmm_encode_only")
        return ws

    def multiply_only(self, M, N, K, out, workspace=None, stream=None):
        ws = workspace if workspace is not None else self.workspace(M, N, K, out.device)
        _check(lib().fmm_multiply_only(self._h, _dev_ptr(out), C.c_int64(M), C.c_int64(N), C.c_int64(K),
                                       _dev_ptr(ws), C.c_size_t(ws.numel()), _stream_ptr(stream)), "fmm_multiply_only")
        return out

    def quantized_view(self, M, N, K, term, side):
        vals = [C.c_size_t(), C.c_int64(), C.c_int64(), C.c_size_t(), C.c_int64(), C.c_int64()]
        _check(lib().fmm_quantized_view(self._h, C.c_int64(M), C.c_int64(N), C.c_int64(K), C.c_int(term),
                                        C.c_char(side.encode()), *[C.byref(v) for v in vals]), "fmm_quantized_view")
        return tuple(v.value for v in vals)

    def quantized_operand(self, ws, M, N, K, term, side):
        """Codes and scales of one leaf operand as numpy arrays in the logical layout:
        side 'A': codes (m, k), scales (m, k/blk); side 'B': codes (k, n), scales (k/blk, n).
        In UE8M0 mode `scales` holds the biased exponent bytes (uint8)."""
        qo, qr, qc, so, sr, sc = self.quantized_view(M, N, K, term, side)
        host = ws.cpu().numpy()
        codes = host[qo:qo + qr * qc].reshape(qr, qc)
        if self.scale_mode == SCALE_FP32:
            scales = host[so:so + sr * sc * 4].view(np.float32).reshape(sr, sc)
            if side == "B":
                codes = codes.T
            else:
                # stored [128-k chunk][row][K block of the chunk]
                g = 128 // self.block_k
                scales = scales.reshape(sr, sc // g, g).transpose(1, 0, 2).reshape(sc // g, sr * g)
        else:
            rows, nkb = sr, sc
            tiles = host[so:so + rows * nkb].reshape(nkb // 4, rows // 128, 32, 4, 4)   # [kb/4, r/128, r%32, (r%128)/32, kb%4]
            scales = tiles.transpose(1, 3, 2, 0, 4).reshape(rows, nkb)
            if side == "B":
                codes = codes.T
                scales = scales.T
        return np.ascontiguousarray(codes), np.ascontiguousarray(scales)

    def device_status(self):
        code = C.c_int()
        st = lib().fmm_device_status(self._h, C.byref(code))
        return st, code.value

    def device_status_clear(self):
        _check(lib().fmm_device_status_clear(self._h), "fmm_device_status_clear")

    def selftest_bounded_wait(self, limit_ns, stream=None):
        _check(lib().fmm_selftest_bounded_wait(self._h, C.c_int64(int(limit_ns)), _stream_ptr(stream)),
               "fmm_selftest_bounded_wait")

    def last_launch_count(self):
        n = C.c_int()
        _check(lib().fmm_last_launch_count(self._h, C.byref(n)), "fmm_last_launch_count")
        return n.value


def fmm_ref_gemm_fp64(A, B, out=None, stream=None):
    import torch
    M, K = A.shape
    _, N = B.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.float64, device=A.device)
    _check(lib().fmm_ref_gemm_fp64(_dev_ptr(A), _dev_ptr(B), _dev_ptr(out), C.c_int64(M), C.c_int64(N), C.c_int64(K),
                                   _stream_ptr(stream)), "fmm_ref_gemm_fp64")
    return out


_scratch = {}


def fmm_error_stats(Cm, Cref, out3=None, stream=None):
    """Device tensor [sum (C-Cref)^2, sum Cref^2, max |C-Cref|] (fp64)."""
    import torch
    M, N = Cm.shape
    if out3 is None:
        out3 = torch.empty(3, dtype=torch.float64, device=Cm.device)
    key = str(Cm.device)
    if key not in _scratch:
        _scratch[key] = torch.empty(lib().fmm_error_stats_scratch_bytes(), dtype=torch.uint8, device=Cm.device)
    sc = _scratch[key]
    _check(lib().fmm_error_stats(_dev_ptr(Cm), _dev_ptr(Cref), C.c_int64(M), C.c_int64(N), _dev_ptr(out3),
                                 _dev_ptr(sc), C.c_size_t(sc.numel()), _stream_ptr(stream)), "fmm_error_stats")
    return out3


def fmm_error_stats_noalloc(Cm, Cref, out3, stream=None):
    """fmm_error_stats_noalloc: same statistics, block partials in the library's built-in scratch.
    Nothing is allocated here either: the caller supplies out3 (3 doubles on the device)."""
    M, N = Cm.shape
    _check(lib().fmm_error_stats_noalloc(_dev_ptr(Cm), _dev_ptr(Cref), C.c_int64(M), C.c_int64(N), _dev_ptr(out3),
                                         _stream_ptr(stream)), "fmm_error_stats_noalloc")
    return out3


def rel_frobenius(Cm, Cref):
    s = fmm_error_stats(Cm, Cref).cpu().numpy()
    return float(np.sqrt(s[0] / s[1]))
