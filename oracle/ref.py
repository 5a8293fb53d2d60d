"""ctypes view of the C oracle (``mxfp4_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Argument marshalling only: every step of the method lives in the C file, in
the paper's order.  bf16 tensors travel as ``numpy.uint16`` bit patterns.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = C.CDLL(_build.build())

_u8p = np.ctypeslib.ndpointer(np.uint8, flags="C_CONTIGUOUS")
_i8p = np.ctypeslib.ndpointer(np.int8, flags="C_CONTIGUOUS")
_u16p = np.ctypeslib.ndpointer(np.uint16, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(np.uint32, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")
_i64 = C.c_int64
_u64 = C.c_uint64

_lib.orc_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
_lib.orc_philox4x32_10.restype = None
_lib.orc_sign_vector.argtypes = [_u64, C.c_int, _i8p]
_lib.orc_sign_vector.restype = None
_lib.orc_sr_draw.argtypes = [_u64, C.c_uint32, _u64]
_lib.orc_sr_draw.restype = C.c_uint32
_lib.orc_hadamard.argtypes = [C.c_int, _i8p]
_lib.orc_hadamard.restype = C.c_int
_lib.orc_rht.argtypes = [C.c_void_p, _i64, _i64, _i64, _i64, C.c_int, _u64, _f32p]
_lib.orc_rht.restype = C.c_int
_lib.orc_transform.argtypes = [C.c_void_p, _i64, _i64, _i64, _i64, C.c_int, C.c_void_p, _f32p]
_lib.orc_transform.restype = C.c_int
_lib.orc_e2m1_value.argtypes = [C.c_uint32]
_lib.orc_e2m1_value.restype = C.c_double
_lib.orc_e8m0_from_amax.argtypes = [C.c_float]
_lib.orc_e8m0_from_amax.restype = C.c_uint32
_lib.orc_sr_round.argtypes = [C.c_double, C.c_uint32]
_lib.orc_sr_round.restype = C.c_uint32
_lib.orc_sr16_draw.argtypes = [_u64, C.c_uint32, _u64]
_lib.orc_sr16_draw.restype = C.c_uint32
_lib.orc_sr16_round.argtypes = [C.c_double, C.c_uint32]
_lib.orc_sr16_round.restype = C.c_uint32
_lib.orc_rn_round.argtypes = [C.c_double]
_lib.orc_rn_round.restype = C.c_uint32
_lib.orc_quantize.argtypes = [_f32p, _i64, _i64, C.c_int, _u64, C.c_uint32, _u8p, _u8p]
_lib.orc_quantize.restype = C.c_int
_lib.orc_quantize_rows.argtypes = [_f32p, _i64, _i64, C.c_int, _u64, C.c_uint32, C.c_void_p, _u8p, _u8p]
_lib.orc_quantize_rows.restype = C.c_int
_lib.orc_pack.argtypes = [_u8p, _i64, _u8p]
_lib.orc_pack.restype = None
_lib.orc_dequantize.argtypes = [_u8p, _u8p, _i64, _i64, _f64p]
_lib.orc_dequantize.restype = None
_lib.orc_gemm.argtypes = [_u8p, _u8p, _u8p, _u8p, _i64, _i64, _i64, C.c_double,
                          C.c_void_p, _i64, C.c_void_p, _i64, _f64p]
_lib.orc_gemm.restype = None
_lib.orc_gemm_bf16.argtypes = [C.c_void_p, _i64, _i64, C.c_void_p, _i64, _i64, _i64,
                               C.c_void_p, _i64, C.c_void_p, _i64, _f64p]
_lib.orc_gemm_bf16.restype = None
_lib.orc_linear_backward.argtypes = [_u16p, _u16p, _u16p, _i64, _i64, _i64, C.c_int, C.c_int, _u64,
                                     C.c_void_p, _i64, C.c_void_p, _i64,
                                     C.c_void_p, _i64, C.c_void_p, _i64, _f64p, _f64p]
_lib.orc_linear_backward.restype = C.c_int
_lib.orc_bias_grad.argtypes = [_u16p, _i64, _i64, _f64p]
_lib.orc_bias_grad.restype = None
_lib.orc_e4m3_value.argtypes = [C.c_uint32]
_lib.orc_e4m3_value.restype = C.c_double
_lib.orc_e4m3_round.argtypes = [C.c_float]
_lib.orc_e4m3_round.restype = C.c_uint32
_lib.orc_fp8_tensor_scale.argtypes = [_u16p, _i64, _i64, _i64, _i64]
_lib.orc_fp8_tensor_scale.restype = C.c_float
_lib.orc_fp8_quantize.argtypes = [_u16p, _i64, _i64, _i64, _i64, C.c_float, _u8p]
_lib.orc_fp8_quantize.restype = None
_lib.orc_fp8_gemm.argtypes = [_u8p, _u8p, _i64, _i64, _i64, C.c_double, C.c_void_p, _i64, C.c_void_p, _i64, _f64p]
_lib.orc_fp8_gemm.restype = None
_lib.orc_linear_forward_fp8.argtypes = [_u16p, _u16p, _i64, _i64, _i64, C.c_void_p, _i64, C.c_void_p, _i64, _f64p]
_lib.orc_linear_forward_fp8.restype = None
_lib.orc_int4_value.argtypes = [C.c_uint32]
_lib.orc_int4_value.restype = C.c_double
_lib.orc_int4_sr_round.argtypes = [C.c_double, C.c_uint32]
_lib.orc_int4_sr_round.restype = C.c_uint32
_lib.orc_int4_rn_round.argtypes = [C.c_double]
_lib.orc_int4_rn_round.restype = C.c_uint32
_lib.orc_mxint4_quantize_rows.argtypes = [_f32p, _i64, _i64, C.c_int, _u64, C.c_uint32, C.c_void_p, _u8p, _u8p]
_lib.orc_mxint4_quantize_rows.restype = C.c_int
_lib.orc_mxint4_gemm.argtypes = [_u8p, _u8p, _u8p, _u8p, _i64, _i64, _i64, C.c_double, C.c_void_p, _i64, C.c_void_p, _i64, _f64p]
_lib.orc_mxint4_gemm.restype = None
_lib.orc_num_threads.argtypes = []
_lib.orc_num_threads.restype = C.c_int

ROUND_SR = 0
ROUND_RN = 1
ROUND_SR16 = 2      # Algorithm 2 with the 16-bit dither of the second SR reading


def num_threads() -> int:
    return int(_lib.orc_num_threads())


def philox4x32_10(ctr, key):
    out = np.zeros(4, np.uint32)
    _lib.orc_philox4x32_10(np.asarray(ctr, np.uint32), np.asarray(key, np.uint32), out)
    return out


def sign_vector(seed: int, g: int) -> np.ndarray:
    S = np.zeros(g, np.int8)
    _lib.orc_sign_vector(seed, g, S)
    return S


def sr_draw(seed: int, stream_tag: int, i: int) -> int:
    return int(_lib.orc_sr_draw(seed, stream_tag, i))


def hadamard(g: int) -> np.ndarray:
    H = np.zeros((g, g), np.int8)
    if _lib.orc_hadamard(g, H) != 0:
        raise ValueError("g must be a power of two")
    return H


def e2m1_value(code: int) -> float:
    return float(_lib.orc_e2m1_value(code))


def e8m0_from_amax(amax: float) -> int:
    return int(_lib.orc_e8m0_from_amax(float(np.float32(amax))))


def sr_round(w: float, r: int) -> int:
    return int(_lib.orc_sr_round(w, r))


def sr16_draw(seed: int, stream_tag: int, i: int) -> int:
    return int(_lib.orc_sr16_draw(seed, stream_tag, i))


def sr16_round(w: float, R: int) -> int:
    return int(_lib.orc_sr16_round(w, R))


def rn_round(w: float) -> int:
    return int(_lib.orc_rn_round(w))


def _view(x: np.ndarray, transpose: bool):
    """(pointer, R, K, stride_r, stride_k) of a 2-D bf16-bit array, optionally viewed transposed."""
    assert x.dtype == np.uint16 and x.ndim == 2 and x.flags.c_contiguous
    rows, cols = x.shape
    if transpose:
        return x.ctypes.data, cols, rows, 1, cols
    return x.ctypes.data, rows, cols, cols, 1


def rht(x: np.ndarray, g: int, seed: int, transpose: bool = False) -> np.ndarray:
    """Blockwise RHT along the reduction dimension; fp32 [R, K] with K the reduce dim."""
    ptr, R, K, sr, sk = _view(x, transpose)
    y = np.empty((R, K), np.float32)
    if _lib.orc_rht(ptr, R, K, sr, sk, g, seed, y) != 0:
        raise ValueError("bad g / shape")
    return y


def transform(x: np.ndarray, T: np.ndarray, transpose: bool = False) -> np.ndarray:
    """Blockwise transform with a given g x g matrix T (bf16 bits): every g-chunk v of the reduce dim becomes v T."""
    ptr, R, K, sr, sk = _view(x, transpose)
    assert T.dtype == np.uint16 and T.ndim == 2 and T.shape[0] == T.shape[1] and T.flags.c_contiguous
    y = np.empty((R, K), np.float32)
    if _lib.orc_transform(ptr, R, K, sr, sk, T.shape[0], T.ctypes.data, y) != 0:
        raise ValueError("bad g / shape")
    return y


def quantize(y: np.ndarray, rounding: int, seed: int, stream_tag: int, row_ids=None):
    """fp32 pre-quantisation values [R, K] -> (codes [R, K] one per byte, scales [R, K/32]).

    row_ids: when y holds a subset of the rows of a larger operand, their row indices there (they key the SR draws)."""
    y = np.ascontiguousarray(y, np.float32)
    R, K = y.shape
    codes = np.empty((R, K), np.uint8)
    scales = np.empty((R, K // 32), np.uint8)
    rp, _n, _keep = _idx(row_ids)
    if _lib.orc_quantize_rows(y, R, K, rounding, seed, stream_tag, rp, codes, scales) != 0:
        raise ValueError("K must be a multiple of 32")
    return codes, scales


def rht_quantize(x, g, rounding, seed, stream_tag, transpose=False, row_ids=None):
    y = rht(x, g, seed, transpose)
    codes, scales = quantize(y, rounding, seed, stream_tag, row_ids)
    return y, codes, scales


def pack(codes: np.ndarray) -> np.ndarray:
    R, K = codes.shape
    out = np.empty((R, K // 2), np.uint8)
    _lib.orc_pack(np.ascontiguousarray(codes), R * K, out)
    return out


def dequantize(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    R, K = codes.shape
    out = np.empty((R, K), np.float64)
    _lib.orc_dequantize(np.ascontiguousarray(codes), np.ascontiguousarray(scales), R, K, out)
    return out


def _idx(a):
    if a is None:
        return None, 0, None
    arr = np.ascontiguousarray(a, np.int64)
    return arr.ctypes.data, arr.size, arr


def gemm(A_codes, A_scales, B_codes, B_scales, alpha=1.0, rows=None, cols=None) -> np.ndarray:
    """C = alpha * deq(A) deq(B)^T in fp64 on the selected rows / cols (None = all)."""
    M, K = A_codes.shape
    N, K2 = B_codes.shape
    assert K == K2
    rp, nr, _r = _idx(rows)
    cp, nc, _c = _idx(cols)
    out = np.empty((nr if rows is not None else M, nc if cols is not None else N), np.float64)
    _lib.orc_gemm(np.ascontiguousarray(A_codes), np.ascontiguousarray(A_scales),
                  np.ascontiguousarray(B_codes), np.ascontiguousarray(B_scales),
                  M, N, K, alpha, rp, nr, cp, nc, out)
    return out


def gemm_bf16(A, B, rows=None, cols=None, a_transpose=False, b_transpose=False) -> np.ndarray:
    """fp64 product C[i, j] = sum_k A(i, k) B(j, k) of bf16 inputs (optionally viewed transposed)."""
    ap, M, K, asr, ask = _view(A, a_transpose)
    bp, N, K2, bsr, bsk = _view(B, b_transpose)
    assert K == K2
    rows = np.arange(M) if rows is None else rows
    cols = np.arange(N) if cols is None else cols
    rp, nr, _r = _idx(rows)
    cp, nc, _c = _idx(cols)
    out = np.empty((nr, nc), np.float64)
    _lib.orc_gemm_bf16(ap, asr, ask, bp, bsr, bsk, K, rp, nr, cp, nc, out)
    return out


def bias_grad(dY):
    """dL/db = column sums of bf16 dY [b, m], fp64 (problem statement, Section 2)."""
    b, m = dY.shape
    db = np.empty(m, np.float64)
    _lib.orc_bias_grad(dY, b, m, db)
    return db


def linear_backward(dY, X, W, g, rounding, seed, dx_rows=None, dx_cols=None, dw_rows=None, dw_cols=None):
    """Algorithm 3 on bf16 dY [b, m], X [b, n], W [m, n]; fp64 (dX, dW) on the selected entries."""
    b, m = dY.shape
    b2, n = X.shape
    m2, n2 = W.shape
    assert b == b2 and m == m2 and n == n2
    p = [_idx(a) for a in (dx_rows, dx_cols, dw_rows, dw_cols)]
    dX = np.empty((p[0][1] if dx_rows is not None else b, p[1][1] if dx_cols is not None else n), np.float64)
    dW = np.empty((p[2][1] if dw_rows is not None else m, p[3][1] if dw_cols is not None else n), np.float64)
    rc = _lib.orc_linear_backward(dY, X, W, b, m, n, g, rounding, seed,
                                  p[0][0], p[0][1], p[1][0], p[1][1],
                                  p[2][0], p[2][1], p[3][0], p[3][1], dX, dW)
    if rc != 0:
        raise ValueError("bad g / shape")
    return dX, dW


# ---------------------------------------------------------------- FP8 (E4M3) forward pass (Section 4.1 / supplementary)
def e4m3_value(code: int) -> float:
    return float(_lib.orc_e4m3_value(code))


def e4m3_round(v: float) -> int:
    return int(_lib.orc_e4m3_round(float(np.float32(v))))


def fp8_tensor_scale(x: np.ndarray) -> float:
    """448 / amax of a bf16 tensor (fp32), 1 for an all-zero tensor."""
    assert x.dtype == np.uint16 and x.ndim == 2 and x.flags.c_contiguous
    return float(_lib.orc_fp8_tensor_scale(x, x.shape[0], x.shape[1], x.shape[1], 1))


def fp8_quantize(x: np.ndarray, scale=None):
    """bf16 [R, K] -> (E4M3 codes [R, K], scale)."""
    if scale is None:
        scale = fp8_tensor_scale(x)
    codes = np.empty(x.shape, np.uint8)
    _lib.orc_fp8_quantize(x, x.shape[0], x.shape[1], x.shape[1], 1, scale, codes)
    return codes, scale


def fp8_gemm(A, B, alpha=1.0, rows=None, cols=None) -> np.ndarray:
    M, K = A.shape
    N, K2 = B.shape
    assert K == K2
    rp, nr, _r = _idx(rows)
    cp, nc, _c = _idx(cols)
    out = np.empty((nr if rows is not None else M, nc if cols is not None else N), np.float64)
    _lib.orc_fp8_gemm(np.ascontiguousarray(A), np.ascontiguousarray(B), M, N, K, alpha, rp, nr, cp, nc, out)
    return out


def linear_forward_fp8(x, W, rows=None, cols=None) -> np.ndarray:
    """y [b, m] = x [b, n] W [m, n]^T with E4M3 operands (one scale per tensor), fp64 accumulation."""
    b, n = x.shape
    m, n2 = W.shape
    assert n == n2
    rp, nr, _r = _idx(rows)
    cp, nc, _c = _idx(cols)
    out = np.empty((nr if rows is not None else b, nc if cols is not None else m), np.float64)
    _lib.orc_linear_forward_fp8(x, W, b, n, m, rp, nr, cp, nc, out)
    return out


# ---------------------------------------------------------------- MXINT4 elements (Section 3, opening remark)
def int4_value(code: int) -> float:
    return float(_lib.orc_int4_value(code))


def int4_sr_round(w: float, r: int) -> int:
    return int(_lib.orc_int4_sr_round(w, r))


def int4_rn_round(w: float) -> int:
    return int(_lib.orc_int4_rn_round(w))


def mxint4_quantize(y: np.ndarray, rounding: int, seed: int, stream_tag: int, row_ids=None):
    """fp32 [R, K] -> (codes [R, K]: bit 3 sign, bits 0-2 magnitude; E8M0 scale bytes [R, K/32])."""
    y = np.ascontiguousarray(y, np.float32)
    R, K = y.shape
    codes = np.empty((R, K), np.uint8)
    scales = np.empty((R, K // 32), np.uint8)
    rp, _n, _keep = _idx(row_ids)
    if _lib.orc_mxint4_quantize_rows(y, R, K, rounding, seed, stream_tag, rp, codes, scales) != 0:
        raise ValueError("K must be a multiple of 32; rounding 0 (SR) or 1 (RN)")
    return codes, scales


def mxint4_gemm(A_codes, A_scales, B_codes, B_scales, alpha=1.0, rows=None, cols=None) -> np.ndarray:
    M, K = A_codes.shape
    N, K2 = B_codes.shape
    assert K == K2
    rp, nr, _r = _idx(rows)
    cp, nc, _c = _idx(cols)
    out = np.empty((nr if rows is not None else M, nc if cols is not None else N), np.float64)
    _lib.orc_mxint4_gemm(np.ascontiguousarray(A_codes), np.ascontiguousarray(A_scales), np.ascontiguousarray(B_codes),
                         np.ascontiguousarray(B_scales), M, N, K, alpha, rp, nr, cp, nc, out)
    return out
