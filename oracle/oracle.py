"""ctypes binding of the CPU oracle (TEST INFRASTRUCTURE ONLY; never on the product path).

Every function takes and returns numpy arrays; the arithmetic lives in
fmm_oracle.c (block quantizer, fused fast matmul, fp64 reference: Sec. 2, App. D.1, App. E.2).
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

SCALE_FP32, SCALE_UE8M0, SCALE_IDENTITY = 0, 1, 2
AMAX_FLOOR = np.float32(1e-12)

_lib = None


def lib():
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        L.oracle_e4m3_encode.restype = C.c_uint8
        L.oracle_e4m3_encode.argtypes = [C.c_float]
        L.oracle_e4m3_decode.restype = C.c_double
        L.oracle_e4m3_decode.argtypes = [C.c_uint8]
        L.oracle_fused_fmm.restype = C.c_int
        L.oracle_encode.restype = C.c_int
        L.oracle_fused_fmm_ex.restype = C.c_int
        L.oracle_encode_ex.restype = C.c_int
        L.oracle_bf16_round.restype = C.c_float
        L.oracle_bf16_round.argtypes = [C.c_float]
        L.oracle_num_threads.restype = C.c_int
        _lib = L
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def _f32(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float32))


def e4m3_encode(y):
    y = np.ascontiguousarray(np.asarray(y, dtype=np.float32))
    out = np.empty(y.shape, dtype=np.uint8)
    lib().oracle_e4m3_encode_array(_p(y), C.c_int64(y.size), _p(out))
    return out


def e4m3_decode(c):
    c = np.ascontiguousarray(np.asarray(c, dtype=np.uint8))
    out = np.empty(c.shape, dtype=np.float64)
    lib().oracle_e4m3_decode_array(_p(c), C.c_int64(c.size), _p(out))
    return out


def dequant_rows(codes, scales, blk):
    """Exact fp64 values of an A-side quantized operand (codes r x c, scales r x c/blk)."""
    return e4m3_decode(codes) * np.repeat(scales.astype(np.float64), blk, axis=1)


def dequant_cols(codes, scales, blk):
    """Exact fp64 values of a B-side quantized operand (codes r x c, scales r/blk x c)."""
    return e4m3_decode(codes) * np.repeat(scales.astype(np.float64), blk, axis=0)


def quant_rows(X, blk, mode=SCALE_FP32, amax_floor=AMAX_FLOOR):
    """A-side quantizer: 1 x blk groups along the columns.  Returns codes, scales, e8."""
    X = _f32(X)
    r, c = X.shape
    codes = np.empty((r, c), np.uint8)
    scales = np.empty((r, c // blk), np.float32)
    e8 = np.empty((r, c // blk), np.uint8)
    lib().oracle_quant_rows(_p(X), C.c_int64(r), C.c_int64(c), C.c_int64(c), C.c_int(blk),
                            C.c_int(mode), C.c_float(float(amax_floor)), _p(codes), _p(scales), _p(e8))
    return codes, scales, e8


def quant_cols(X, blk, mode=SCALE_FP32, amax_floor=AMAX_FLOOR):
    """B-side quantizer: blk x 1 groups along the rows.  Returns codes, scales, e8."""
    X = _f32(X)
    r, c = X.shape
    codes = np.empty((r, c), np.uint8)
    scales = np.empty((r // blk, c), np.float32)
    e8 = np.empty((r // blk, c), np.uint8)
    lib().oracle_quant_cols(_p(X), C.c_int64(r), C.c_int64(c), C.c_int64(c), C.c_int(blk),
                            C.c_int(mode), C.c_float(float(amax_floor)), _p(codes), _p(scales), _p(e8))
    return codes, scales, e8


def quant_tiles(X, blk, tile, amax_floor=AMAX_FLOOR):
    """B-side quantizer with one FP32 scale per blk x tile tile (App. E.5); shapes as quant_cols."""
    X = _f32(X)
    rows, cols = X.shape
    codes = np.empty((rows, cols), np.uint8)
    scales = np.empty((rows // blk, cols), np.float32)
    lib().oracle_quant_tiles(_p(X), C.c_int64(rows), C.c_int64(cols), C.c_int64(cols), C.c_int(blk), C.c_int(tile),
                             C.c_float(float(amax_floor)), _p(codes), _p(scales))
    return codes, scales


def bf16_round(x):
    """Elementwise round-to-nearest-even to bfloat16, widened back to fp32."""
    x = _f32(np.atleast_1d(x))
    f = lib().oracle_bf16_round
    return np.array([f(float(v)) for v in x.ravel()], np.float32).reshape(x.shape)


def _uvw(U, V, W):
    U = _f32(U) if U is not None else None
    V = _f32(V) if V is not None else None
    W = _f32(W) if W is not None else None
    return U, V, W


def fused_fmm(A, B, U=None, V=None, W=None, levels=1, blk=32, mode=SCALE_FP32,
              amax_floor=AMAX_FLOOR, b_tile=0, b_bf16=False):
    """C (fp64) of the fused block-scaled fast product; levels=0 is cubic fp8.
    b_tile / b_bf16: the weight-side options of App. E.5 (blk x b_tile scale tiles, bf16 pre-round)."""
    A, B = _f32(A), _f32(B)
    M, K = A.shape
    K2, N = B.shape
    assert K == K2
    U, V, W = _uvw(U, V, W)
    rank = 0 if U is None else U.shape[0]
    Cout = np.empty((M, N), np.float64)
    rc = lib().oracle_fused_fmm_ex(_p(A), _p(B), _p(Cout), C.c_int64(M), C.c_int64(N), C.c_int64(K),
                                   C.c_int(rank), _p(U) if U is not None else None,
                                   _p(V) if V is not None else None, _p(W) if W is not None else None,
                                   C.c_int(levels), C.c_int(blk), C.c_int(mode),
                                   C.c_float(float(amax_floor)), C.c_int(int(b_tile)), C.c_int(int(bool(b_bf16))))
    if rc:
        raise ValueError(f"oracle_fused_fmm rejected the arguments (code {rc})")
    return Cout


def encode(X, side, U, V, levels, blk=32, mode=SCALE_FP32, amax_floor=AMAX_FLOOR, b_tile=0, b_bf16=False):
    """Quantized leaf operands of one side ('A' or 'B'), depth-first term order.
    'A': codes [T, m, k], scales [T, m, k/blk];  'B': codes [T, k, n], scales [T, k/blk, n]."""
    X = _f32(X)
    rows, cols = X.shape
    U, V, _ = _uvw(U, V, None)
    rank = 1 if U is None else U.shape[0]
    T = rank ** levels if levels > 0 else 1
    d = 1 << levels
    lr, lc = rows // d, cols // d
    s = 0 if side == "A" else 1
    codes = np.empty((T, lr, lc), np.uint8)
    sshape = (T, lr, lc // blk) if s == 0 else (T, lr // blk, lc)
    scales = np.empty(sshape, np.float32)
    e8 = np.empty(sshape, np.uint8)
    rc = lib().oracle_encode_ex(_p(X), C.c_int64(rows), C.c_int64(cols), C.c_int(s), C.c_int(rank),
                                _p(U) if U is not None else None, _p(V) if V is not None else None,
                                C.c_int(levels), C.c_int(blk), C.c_int(mode),
                                C.c_float(float(amax_floor)), C.c_int(int(b_tile)), C.c_int(int(bool(b_bf16))),
                                _p(codes), _p(scales), _p(e8))
    if rc:
        raise ValueError(f"oracle_encode rejected the arguments (code {rc})")
    return codes, scales, e8


def ref_gemm(A, B):
    """fp64 product of the fp32 inputs (App. E.2's reference), plain loops."""
    A, B = _f32(A), _f32(B)
    M, K = A.shape
    _, N = B.shape
    Cout = np.empty((M, N), np.float64)
    lib().oracle_ref_gemm(_p(A), _p(B), _p(Cout), C.c_int64(M), C.c_int64(N), C.c_int64(K))
    return Cout


def ref_gemm_rows(A, B, rows):
    A, B = _f32(A), _f32(B)
    M, K = A.shape
    _, N = B.shape
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    out = np.empty((rows.size, N), np.float64)
    lib().oracle_ref_gemm_rows(_p(A), _p(B), _p(rows), C.c_int64(rows.size), _p(out),
                               C.c_int64(M), C.c_int64(N), C.c_int64(K))
    return out


def leaf_product_sample(codes_a, scales_a, codes_b, scales_b, blk, rows, cols):
    """Entries (rows x cols) of one leaf product S^ T^ in fp64 from the quantized operands of one term as
    `encode` returns them (A side [m, k] / [m, k/blk], B side [k, n] / [k/blk, n]); plain loops in C."""
    ca = np.ascontiguousarray(codes_a, dtype=np.uint8)
    cb = np.ascontiguousarray(codes_b, dtype=np.uint8)
    sa, sb = _f32(scales_a), _f32(scales_b)
    m, k = ca.shape
    k2, n = cb.shape
    assert k == k2 and sa.shape == (m, k // blk) and sb.shape == (k // blk, n)
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    cols = np.ascontiguousarray(np.asarray(cols, dtype=np.int64))
    out = np.empty((rows.size, cols.size), np.float64)
    lib().oracle_leaf_product_sample(_p(ca), _p(sa), _p(cb), _p(sb), C.c_int64(m), C.c_int64(n), C.c_int64(k),
                                     C.c_int(blk), _p(rows), C.c_int64(rows.size), _p(cols), C.c_int64(cols.size),
                                     _p(out))
    return out


def error_stats(Cm, Cref):
    """[sum (C-Cref)^2, sum Cref^2, max |C-Cref|] in fp64."""
    Cm = np.ascontiguousarray(np.asarray(Cm, dtype=np.float64))
    Cref = np.ascontiguousarray(np.asarray(Cref, dtype=np.float64))
    out = np.empty(3, np.float64)
    lib().oracle_error_stats(_p(Cm), _p(Cref), C.c_int64(Cm.size), _p(out))
    return out


def rel_frobenius(Cm, Cref):
    s = error_stats(Cm, Cref)
    return float(np.sqrt(s[0] / s[1]))


def num_threads():
    return int(lib().oracle_num_threads())
