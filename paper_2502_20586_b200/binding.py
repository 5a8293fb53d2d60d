"""Thin Python binding of the C-ABI library (include/mxfp4.h): argument marshalling only.

Every step of the method runs in the CUDA kernels behind ``libmxfp4_b200.so``; torch is used for device
memory and streams.  There is no CPU fallback: if the library has not been built this module fails to import.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmxfp4_b200.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2502_20586_b200.build` "
                      "(there is no CPU fallback)")
_lib = C.CDLL(LIB_PATH)

OK = 0
ROUND_SR, ROUND_RN, ROUND_SR16 = 0, 1, 2
SF_LINEAR, SF_NATIVE = 0, 1
OUT_BF16, OUT_FP32 = 0, 1

_vp, _i64, _u64, _u32, _int, _sz = C.c_void_p, C.c_int64, C.c_uint64, C.c_uint32, C.c_int, C.c_size_t
_lib.mxfp4_rht_sr_quantize.argtypes = [_vp, _i64, _i64, _i64, _int, _int, _int, _u64, _u32, _vp, _vp, _int, _vp]
_lib.mxfp4_rht_sr_quantize.restype = _int
_lib.mxfp4_transform_quantize.argtypes = [_vp, _i64, _i64, _i64, _int, _int, _vp, _int, _u64, _u32, _vp, _vp, _int, _vp, _vp]
_lib.mxfp4_transform_quantize.restype = _int
_lib.mxfp4_rht.argtypes = [_vp, _i64, _i64, _i64, _int, _int, _u64, _vp, _vp]
_lib.mxfp4_rht.restype = _int
_lib.mxfp4_gemm.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _int, C.c_float, _vp, _i64, _int, _vp]
_lib.mxfp4_gemm.restype = _int
_lib.mxfp4_linear_backward_workspace.argtypes = [_i64, _i64, _i64]
_lib.mxfp4_linear_backward_workspace.restype = _sz
_lib.mxfp4_linear_backward.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _int, _int, _u64, _vp, _vp, _int, _vp, _sz, _vp]
_lib.mxfp4_linear_backward.restype = _int
_lib.mxfp4_linear_backward_static.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _int, _int, _u64, _vp, _vp, _int, _vp]
_lib.mxfp4_linear_backward_static.restype = _int
_lib.mxfp4_linear_backward_ex_workspace.argtypes = [_i64, _i64, _i64, _int]
_lib.mxfp4_linear_backward_ex_workspace.restype = _sz
_lib.mxfp4_linear_backward_ex.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _int, _int, _u64, _vp, _vp, _vp, _int, _int, _vp, _sz, _vp]
_lib.mxfp4_linear_backward_ex.restype = _int
_lib.mxfp4_gemm_fused.argtypes = [_vp, _i64, _i64, _i64, _int, _int, _int, _u64, _u32, _vp, _vp, _i64, C.c_float, _vp, _i64, _int, _vp]
_lib.mxfp4_gemm_fused.restype = _int
_lib.mxfp4_linear_backward_fused.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _int, _int, _u64, _vp, _vp, _int, _vp, _sz, _vp]
_lib.mxfp4_linear_backward_fused.restype = _int
_lib.mxfp4_operand_layout.argtypes = [_i64, _i64, _i64, C.POINTER(_sz)]
_lib.mxfp4_operand_layout.restype = None
_lib.mxfp4_quantize_operands.argtypes = [_vp, _vp, _vp, _i64, _i64, _i64, _int, _int, _u64, _vp, _sz, _vp]
_lib.mxfp4_quantize_operands.restype = _int
_lib.mxfp4_selftest_wait_expiry.argtypes = [_vp]
_lib.mxfp4_selftest_wait_expiry.restype = _int
_lib.mxfp4_fp4_ceiling.argtypes = [_i64, C.POINTER(C.c_int64), _vp]
_lib.mxfp4_fp4_ceiling.restype = _int
_lib.mxfp4_fp8_quantize.argtypes = [_vp, _i64, _i64, _i64, _vp, _vp, _vp]
_lib.mxfp4_fp8_quantize.restype = _int
_lib.mxfp4_fp8_gemm.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _i64, _int, _vp]
_lib.mxfp4_fp8_gemm.restype = _int
_lib.mxfp4_linear_forward_fp8_workspace.argtypes = [_i64, _i64, _i64]
_lib.mxfp4_linear_forward_fp8_workspace.restype = _sz
_lib.mxfp4_linear_forward_fp8.argtypes = [_vp, _vp, _i64, _i64, _i64, _vp, _int, _vp, _sz, _vp]
_lib.mxfp4_linear_forward_fp8.restype = _int
_lib.mxfp4_int4_quantize.argtypes = [_vp, _i64, _i64, _i64, _int, _int, _int, _u64, _u32, _vp, _vp, _vp, _vp]
_lib.mxfp4_int4_quantize.restype = _int
_lib.mxfp4_int4_gemm.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _i64, C.c_float, _vp, _i64, _int, _vp]
_lib.mxfp4_int4_gemm.restype = _int
_lib.mxfp4_scale_bytes.argtypes = [_i64, _i64, _int]
_lib.mxfp4_scale_bytes.restype = _sz
_lib.mxfp4_device_status.argtypes = [_vp]
_lib.mxfp4_device_status.restype = _int
_lib.mxfp4_status_string.argtypes = [_int]
_lib.mxfp4_status_string.restype = C.c_char_p

EXPORTS = ["mxfp4_rht_sr_quantize", "mxfp4_rht", "mxfp4_gemm", "mxfp4_linear_backward_workspace",
           "mxfp4_linear_backward", "mxfp4_linear_backward_static", "mxfp4_scale_bytes", "mxfp4_device_status", "mxfp4_status_string",
           "mxfp4_fp4_ceiling", "mxfp4_linear_backward_ex_workspace", "mxfp4_linear_backward_ex", "mxfp4_gemm_fused",
           "mxfp4_linear_backward_fused", "mxfp4_operand_layout", "mxfp4_quantize_operands", "mxfp4_transform_quantize",
           "mxfp4_selftest_wait_expiry", "mxfp4_fp8_quantize", "mxfp4_fp8_gemm", "mxfp4_linear_forward_fp8_workspace",
           "mxfp4_linear_forward_fp8", "mxfp4_int4_quantize", "mxfp4_int4_gemm"]


class MxFp4Error(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(f"mxfp4 error {code}: {_lib.mxfp4_status_string(code).decode()}")


def _check(code: int):
    if code != OK:
        raise MxFp4Error(code)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def lib():
    """The raw ctypes handle (tests use it to probe error codes with arbitrary arguments)."""
    return _lib


def mxfp4_selftest_wait_expiry() -> None:
    """Launch the diagnostic kernel whose bounded wait expires (about two seconds); the next device status is TIMEOUT."""
    _check(_lib.mxfp4_selftest_wait_expiry(_stream()))


def mxfp4_scale_bytes(rows: int, K: int, sf_layout: int = SF_NATIVE) -> int:
    return int(_lib.mxfp4_scale_bytes(rows, K, sf_layout))


def mxfp4_rht_sr_quantize(x: torch.Tensor, reduce_dim: int, g: int, seed: int, stream_tag: int = 0,
                          rounding: int = ROUND_SR, sf_layout: int = SF_NATIVE, codes=None, scales=None):
    """x: bf16 [rows, cols] on the GPU (row stride = x.stride(0)).  Returns (codes [R, K/2] u8, scales u8 flat)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    R, K = (rows, cols) if reduce_dim == 1 else (cols, rows)
    if codes is None:
        codes = torch.empty((R, K // 2), dtype=torch.uint8, device=x.device)
    if scales is None:
        scales = torch.empty(mxfp4_scale_bytes(R, K, sf_layout), dtype=torch.uint8, device=x.device)
    _check(_lib.mxfp4_rht_sr_quantize(_ptr(x), rows, cols, x.stride(0), reduce_dim, g, rounding, seed, stream_tag,
                                      _ptr(codes), _ptr(scales), sf_layout, _stream()))
    return codes, scales


def mxfp4_rht(x: torch.Tensor, reduce_dim: int, g: int, seed: int, y=None):
    """The transform alone: fp32 [R, K] with K the reduction dimension."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    R, K = (rows, cols) if reduce_dim == 1 else (cols, rows)
    if y is None:
        y = torch.empty((R, K), dtype=torch.float32, device=x.device)
    _check(_lib.mxfp4_rht(_ptr(x), rows, cols, x.stride(0), reduce_dim, g, seed, _ptr(y), _stream()))
    return y


def mxfp4_transform_quantize(x, reduce_dim: int, T, seed: int, stream_tag: int = 0, rounding: int = ROUND_SR,
                             sf_layout: int = SF_NATIVE, dump: bool = False):
    """Quantiser with a caller-given transform matrix T (bf16 [g, g]): (codes, scales), or the fp32 transform if dump."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    assert T.is_cuda and T.dtype == torch.bfloat16 and T.dim() == 2 and T.shape[0] == T.shape[1] and T.is_contiguous()
    rows, cols = x.shape
    R, K = (rows, cols) if reduce_dim == 1 else (cols, rows)
    g = T.shape[0]
    if dump:
        y = torch.empty((R, K), dtype=torch.float32, device=x.device)
        _check(_lib.mxfp4_transform_quantize(_ptr(x), rows, cols, x.stride(0), reduce_dim, g, _ptr(T), rounding, seed, stream_tag,
                                             0, 0, sf_layout, _ptr(y), _stream()))
        return y
    codes = torch.empty((R, K // 2), dtype=torch.uint8, device=x.device)
    scales = torch.empty(mxfp4_scale_bytes(R, K, sf_layout), dtype=torch.uint8, device=x.device)
    _check(_lib.mxfp4_transform_quantize(_ptr(x), rows, cols, x.stride(0), reduce_dim, g, _ptr(T), rounding, seed, stream_tag,
                                         _ptr(codes), _ptr(scales), sf_layout, 0, _stream()))
    return codes, scales


def mxfp4_gemm(A_codes, A_scales, B_codes, B_scales, alpha: float = 1.0, out_dtype: int = OUT_BF16, C_out=None):
    """C[M, N] = alpha * deq(A) deq(B)^T; codes [M, K/2] / [N, K/2] u8, scales in the native layout."""
    M, K2 = A_codes.shape
    N, K2b = B_codes.shape
    assert K2 == K2b
    if C_out is None:
        C_out = torch.empty((M, N), dtype=torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16, device=A_codes.device)
    _check(_lib.mxfp4_gemm(_ptr(A_codes), _ptr(A_scales), _ptr(B_codes), _ptr(B_scales), M, N, 2 * K2, SF_NATIVE,
                           alpha, _ptr(C_out), C_out.stride(0), out_dtype, _stream()))
    return C_out


def mxfp4_gemm_fused(x, reduce_dim: int, g: int, seed: int, stream_tag: int, rounding: int, B_codes, B_scales,
                     alpha: float = 1.0, out_dtype: int = OUT_BF16, C_out=None):
    """C = alpha * Q(RHT(A)) deq(B)^T with A = x (reduce_dim 1) or x^T (reduce_dim 0) quantised inside the GEMM kernel."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    M = rows if reduce_dim == 1 else cols
    N = B_codes.shape[0]
    if C_out is None:
        C_out = torch.empty((M, N), dtype=torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16, device=x.device)
    _check(_lib.mxfp4_gemm_fused(_ptr(x), rows, cols, x.stride(0), reduce_dim, g, rounding, seed, stream_tag, _ptr(B_codes),
                                 _ptr(B_scales), N, alpha, _ptr(C_out), C_out.stride(0), out_dtype, _stream()))
    return C_out


def mxfp4_linear_backward_fused(dY, X, W, g: int, seed: int, rounding: int = ROUND_SR, out_dtype: int = OUT_BF16,
                                dX=None, dW=None, workspace=None):
    """Algorithm 3 with dY / dY^T transformed and quantised inside the two GEMM kernels (fused-producer variant)."""
    b, m = dY.shape
    _, n = X.shape
    for t in (dY, X, W):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
    dt = torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16
    if dX is None:
        dX = torch.empty((b, n), dtype=dt, device=dY.device)
    if dW is None:
        dW = torch.empty((m, n), dtype=dt, device=dY.device)
    if workspace is None:
        workspace = torch.empty(mxfp4_linear_backward_workspace(b, m, n), dtype=torch.uint8, device=dY.device)
    _check(_lib.mxfp4_linear_backward_fused(_ptr(dY), _ptr(X), _ptr(W), b, m, n, g, rounding, seed, _ptr(dX), _ptr(dW),
                                            out_dtype, _ptr(workspace), workspace.numel(), _stream()))
    return dX, dW


def mxfp4_quantize_operands(dY, X, W, g: int, seed: int, rounding: int = ROUND_SR, workspace=None):
    """Algorithm 3 lines 3-6 in one launch.  Returns [(codes, scales)] for Q1..Q4 as views into the workspace
    (codes [R, K/2] u8, scales flat u8 in the native layout), ready for mxfp4_gemm."""
    b, m = dY.shape
    _, n = X.shape
    for t in (dY, X, W):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
    if workspace is None:
        workspace = torch.empty(mxfp4_linear_backward_workspace(b, m, n), dtype=torch.uint8, device=dY.device)
    _check(_lib.mxfp4_quantize_operands(_ptr(dY), _ptr(X), _ptr(W), b, m, n, g, rounding, seed, _ptr(workspace), workspace.numel(),
                                        _stream()))
    off = (_sz * 8)()
    _lib.mxfp4_operand_layout(b, m, n, off)
    shapes = ((b, m), (n, m), (m, b), (n, b))
    out = []
    for i, (R, K) in enumerate(shapes):
        codes = workspace[off[2 * i]: off[2 * i] + R * K // 2].view(R, K // 2)
        scales = workspace[off[2 * i + 1]: off[2 * i + 1] + mxfp4_scale_bytes(R, K)]
        out.append((codes, scales))
    return out


def mxfp4_operand_layout(b: int, m: int, n: int):
    """Byte offsets [(codes, scales)] x 4 of the quantised operands Q1..Q4 inside a backward workspace."""
    off = (_sz * 8)()
    _lib.mxfp4_operand_layout(b, m, n, off)
    return [(int(off[2 * i]), int(off[2 * i + 1])) for i in range(4)]


def mxfp4_linear_backward_workspace(b: int, m: int, n: int) -> int:
    return int(_lib.mxfp4_linear_backward_workspace(b, m, n))


def mxfp4_linear_backward(dY, X, W, g: int, seed: int, rounding: int = ROUND_SR, out_dtype: int = OUT_BF16,
                          dX=None, dW=None, workspace=None):
    """Algorithm 3: dY [b, m], X [b, n], W [m, n] bf16 (contiguous)  ->  (dX [b, n], dW [m, n])."""
    b, m = dY.shape
    _, n = X.shape
    for t in (dY, X, W):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
    dt = torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16
    if dX is None:
        dX = torch.empty((b, n), dtype=dt, device=dY.device)
    if dW is None:
        dW = torch.empty((m, n), dtype=dt, device=dY.device)
    need = mxfp4_linear_backward_workspace(b, m, n)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dY.device)
    _check(_lib.mxfp4_linear_backward(_ptr(dY), _ptr(X), _ptr(W), b, m, n, g, rounding, seed, _ptr(dX), _ptr(dW),
                                      out_dtype, _ptr(workspace), workspace.numel(), _stream()))
    return dX, dW


def mxfp4_linear_backward_ex_workspace(b: int, m: int, n: int, with_bias: bool) -> int:
    return int(_lib.mxfp4_linear_backward_ex_workspace(b, m, n, 1 if with_bias else 0))


def mxfp4_linear_backward_ex(dY, X, W, g: int, seed: int, rounding: int = ROUND_SR, out_dtype: int = OUT_BF16,
                             dX=None, dW=None, db=None, with_bias: bool = False, accumulate: bool = False, workspace=None):
    """Algorithm 3 plus the bias gradient (fp32 [m], column sums of dY) and accumulation into fp32 dW / db.
    Returns (dX, dW, db) with db None unless with_bias or db is given."""
    b, m = dY.shape
    _, n = X.shape
    for t in (dY, X, W):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
    dt = torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16
    if dX is None:
        dX = torch.empty((b, n), dtype=dt, device=dY.device)
    if dW is None:
        assert not accumulate, "accumulation needs an existing dW"
        dW = torch.empty((m, n), dtype=dt, device=dY.device)
    if db is None and with_bias:
        assert not accumulate, "accumulation needs an existing db"
        db = torch.empty((m,), dtype=torch.float32, device=dY.device)
    need = mxfp4_linear_backward_ex_workspace(b, m, n, db is not None)
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=dY.device)
    _check(_lib.mxfp4_linear_backward_ex(_ptr(dY), _ptr(X), _ptr(W), b, m, n, g, rounding, seed, _ptr(dX), _ptr(dW),
                                         _ptr(db) if db is not None else None, out_dtype, 1 if accumulate else 0,
                                         _ptr(workspace), workspace.numel(), _stream()))
    return dX, dW, db


STATIC_WORKSPACE_BYTES = 8 << 20


def mxfp4_linear_backward_static(dY, X, W, g: int, seed: int, rounding: int = ROUND_SR, out_dtype: int = OUT_BF16,
                                 dX=None, dW=None):
    """mxfp4_linear_backward for callers that cannot provide scratch memory: the library's own fixed array
    (STATIC_WORKSPACE_BYTES per GPU) holds the quantised operands.  Pass dX and dW to make the call itself
    allocation-free; shapes that need more scratch than the array raise MxFp4Error(6)."""
    b, m = dY.shape
    _, n = X.shape
    for t in (dY, X, W):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
    dt = torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16
    if dX is None:
        dX = torch.empty((b, n), dtype=dt, device=dY.device)
    if dW is None:
        dW = torch.empty((m, n), dtype=dt, device=dY.device)
    _check(_lib.mxfp4_linear_backward_static(_ptr(dY), _ptr(X), _ptr(W), b, m, n, g, rounding, seed, _ptr(dX), _ptr(dW),
                                             out_dtype, _stream()))
    return dX, dW


def mxfp4_fp4_ceiling(mma_per_pair: int) -> int:
    """Launches the tensor-pipe ceiling kernel on the current stream and returns the flop it performs (time it with events)."""
    flop = C.c_int64(0)
    _check(_lib.mxfp4_fp4_ceiling(mma_per_pair, C.byref(flop), _stream()))
    return int(flop.value)


def mxfp4_device_status() -> int:
    """Synchronises the current stream and returns the status code (0 = OK, 9 = a device-side wait timed out)."""
    return int(_lib.mxfp4_device_status(_stream()))


# ---------------------------------------------------------------- FP8 (E4M3) forward pass
def mxfp4_fp8_quantize(x: torch.Tensor, codes=None, scale=None):
    """x bf16 [rows, cols] -> (E4M3 codes [rows, cols] u8, scale f32[2] on the device: 448 / amax, amax)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    if codes is None:
        codes = torch.empty((rows, cols), dtype=torch.uint8, device=x.device)
    if scale is None:
        scale = torch.empty(2, dtype=torch.float32, device=x.device)
    _check(_lib.mxfp4_fp8_quantize(_ptr(x), rows, cols, x.stride(0), _ptr(codes), _ptr(scale), _stream()))
    return codes, scale


def mxfp4_fp8_gemm(A_codes, A_scale, B_codes, B_scale, out_dtype: int = OUT_BF16, C_out=None):
    """C [M, N] = A B^T / (A_scale[0] B_scale[0]) with E4M3 operands [M, K], [N, K]."""
    M, K = A_codes.shape
    N = B_codes.shape[0]
    if C_out is None:
        C_out = torch.empty((M, N), dtype=torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16, device=A_codes.device)
    _check(_lib.mxfp4_fp8_gemm(_ptr(A_codes), _ptr(A_scale), _ptr(B_codes), _ptr(B_scale), M, N, K, _ptr(C_out), C_out.stride(0),
                               out_dtype, _stream()))
    return C_out


def mxfp4_linear_forward_fp8(x, W, out_dtype: int = OUT_BF16, y=None, workspace=None):
    """y [b, m] = x [b, n] W [m, n]^T through E4M3 (one scale per tensor)."""
    b, n = x.shape
    m = W.shape[0]
    for t in (x, W):
        assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()
    if y is None:
        y = torch.empty((b, m), dtype=torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16, device=x.device)
    if workspace is None:
        workspace = torch.empty(int(_lib.mxfp4_linear_forward_fp8_workspace(b, n, m)), dtype=torch.uint8, device=x.device)
    _check(_lib.mxfp4_linear_forward_fp8(_ptr(x), _ptr(W), b, n, m, _ptr(y), out_dtype, _ptr(workspace), workspace.numel(), _stream()))
    return y


# ---------------------------------------------------------------- MXINT4 elements
def mxfp4_int4_quantize(x: torch.Tensor, reduce_dim: int, g: int, seed: int, stream_tag: int = 0, rounding: int = ROUND_SR):
    """x bf16 [rows, cols] -> (codes [R, K] u8: the integers -7..7 as E4M3 bytes, scales u8 in the native layout,
    y fp32 [R, K]: the transformed values that were rounded)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    rows, cols = x.shape
    R, K = (rows, cols) if reduce_dim == 1 else (cols, rows)
    codes = torch.empty((R, K), dtype=torch.uint8, device=x.device)
    scales = torch.zeros(mxfp4_scale_bytes(R, K, SF_NATIVE), dtype=torch.uint8, device=x.device)
    y = torch.empty((R, K), dtype=torch.float32, device=x.device)
    _check(_lib.mxfp4_int4_quantize(_ptr(x), rows, cols, x.stride(0), reduce_dim, g, rounding, seed, stream_tag, _ptr(codes), _ptr(scales),
                                    _ptr(y), _stream()))
    return codes, scales, y


def mxfp4_int4_gemm(A_codes, A_scales, B_codes, B_scales, alpha: float = 1.0, out_dtype: int = OUT_BF16, C_out=None):
    """C [M, N] = alpha * sum_k (q X)_A (q X)_B for MXINT4 operands [M, K], [N, K] (one byte per element)."""
    M, K = A_codes.shape
    N = B_codes.shape[0]
    if C_out is None:
        C_out = torch.empty((M, N), dtype=torch.float32 if out_dtype == OUT_FP32 else torch.bfloat16, device=A_codes.device)
    _check(_lib.mxfp4_int4_gemm(_ptr(A_codes), _ptr(A_scales), _ptr(B_codes), _ptr(B_scales), M, N, K, alpha, _ptr(C_out), C_out.stride(0),
                                out_dtype, _stream()))
    return C_out
