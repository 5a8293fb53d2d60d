"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header declares,
and rejects bad arguments with error codes before touching the device."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2502_20586_b200 import build
    build.build()
    from paper_2502_20586_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "mxfp4.h")).read()
    declared = re.findall(r"MXFP4_API\s+[\w\s\*]+?\b(mxfp4_\w+)\s*\(", header)
    assert len(declared) >= 8
    raw = C.CDLL(lib.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name
    assert sorted(declared) == sorted(lib.EXPORTS)


def test_status_strings(lib):
    raw = lib.lib()
    seen = {raw.mxfp4_status_string(i) for i in range(10)}
    assert len(seen) == 10 and b"ok" in seen


def test_scale_bytes_and_workspace(lib):
    assert lib.mxfp4_scale_bytes(256, 512, lib.SF_LINEAR) == 256 * 16
    assert lib.mxfp4_scale_bytes(256, 512, lib.SF_NATIVE) == 2 * 4 * 512
    assert lib.mxfp4_scale_bytes(129, 160, lib.SF_NATIVE) == 2 * 2 * 512          # padded to 128 rows x 4 blocks
    assert lib.mxfp4_scale_bytes(0, 512, lib.SF_NATIVE) == 0
    b, m, n = 256, 512, 512
    need = lib.mxfp4_linear_backward_workspace(b, m, n)
    codes = (b * m + n * m + m * b + n * b) // 2
    assert need >= codes + codes // 16 and need % 256 == 0
    assert lib.mxfp4_linear_backward_workspace(0, m, n) == 0


def test_argument_validation_needs_no_device(lib):
    raw = lib.lib()
    P = 0x1000                                    # a fake, 16-byte aligned, never dereferenced pointer
    q = raw.mxfp4_rht_sr_quantize
    assert q(0, 32, 64, 64, 1, 64, 0, 0, 0, P, P, 1, 0) == 1                      # NULL
    assert q(P, 32, 64, 64, 1, 64, 0, 0, 0, 0, P, 1, 0) == 1
    assert q(P, 0, 64, 64, 1, 64, 0, 0, 0, P, P, 1, 0) == 2                       # shape
    assert q(P, 32, 64, 32, 1, 64, 0, 0, 0, P, P, 1, 0) == 2                      # ld < cols
    assert q(P, 32, 48, 48, 1, 0, 0, 0, 0, P, P, 1, 0) == 2                       # K % 32
    assert q(P, 32, 64, 64, 1, 48, 0, 0, 0, P, P, 1, 0) == 4                      # g not a power of two
    assert q(P, 32, 64, 64, 1, 128, 0, 0, 0, P, P, 1, 0) == 4                     # g does not divide K
    assert q(P, 64, 64, 64, 0, 128, 0, 0, 0, P, P, 1, 0) == 4
    assert q(P, 32, 64, 64, 2, 64, 0, 0, 0, P, P, 1, 0) == 5                      # reduce_dim
    assert q(P, 32, 64, 64, 1, 64, 7, 0, 0, P, P, 1, 0) == 5                      # rounding
    assert q(P, 32, 64, 64, 1, 64, 3, 0, 0, P, P, 1, 0) == 5 and q(P, 32, 64, 64, 1, 64, -1, 0, 0, P, P, 1, 0) == 5
    assert q(P, 32, 64, 64, 1, 64, 0, 0, 0, P, P, 3, 0) == 5                      # layout
    assert q(P + 2, 32, 64, 64, 1, 64, 0, 0, 0, P, P, 1, 0) == 3                  # alignment
    assert q(P, 32, 64, 68, 1, 64, 0, 0, 0, P, P, 1, 0) == 3                      # ld % 8
    g = raw.mxfp4_gemm
    assert g(0, P, P, P, 128, 128, 128, 1, 1.0, P, 128, 0, 0) == 1
    assert g(P, P, P, P, 128, 128, 96, 1, 1.0, P, 128, 0, 0) == 2                 # K % 128
    assert g(P, P, P, P, 128, 100, 128, 1, 1.0, P, 128, 0, 0) == 2                # N % 8
    assert g(P, P, P, P, 128, 128, 128, 1, 1.0, P, 64, 0, 0) == 2                 # ldc < N
    assert g(P, P, P, P, 128, 128, 128, 0, 1.0, P, 128, 0, 0) == 5                # linear scales not accepted
    assert g(P, P, P, P, 128, 128, 128, 1, 1.0, P, 128, 9, 0) == 5
    assert g(P, P, P + 4, P, 128, 128, 128, 1, 1.0, P, 128, 0, 0) == 3
    lb = raw.mxfp4_linear_backward
    assert lb(P, P, 0, 256, 512, 512, 64, 0, 0, P, P, 0, P, 1 << 30, 0) == 1
    assert lb(P, P, P, 256, 500, 512, 64, 0, 0, P, P, 0, P, 1 << 30, 0) == 2
    assert lb(P, P, P, 256, 512, 512, 96, 0, 0, P, P, 0, P, 1 << 30, 0) == 4
    assert lb(P, P, P, 128, 512, 512, 256, 0, 0, P, P, 0, P, 1 << 30, 0) == 4     # g does not divide b
    assert lb(P, P, P, 256, 512, 512, 64, 0, 0, P, P, 0, 0, 1 << 30, 0) == 6      # workspace NULL
    assert lb(P, P, P, 256, 512, 512, 64, 0, 0, P, P, 0, P, 1024, 0) == 6         # too small
    assert lb(P, P, P, 256, 512, 512, 64, 0, 0, P, P, 0, P + 16, 1 << 30, 0) == 6  # misaligned
    # extended form: bias gradient and accumulation
    ex = raw.mxfp4_linear_backward_ex
    big = 1 << 30
    assert ex(P, P, P, 256, 512, 512, 64, 0, 0, P, 0, P, 1, 0, P, big, 0) == 1         # dW NULL
    assert ex(P, P, P, 256, 512, 512, 64, 0, 0, P, P, P, 0, 1, P, big, 0) == 5         # accumulate needs fp32 outputs
    assert ex(P, P, P, 256, 512, 512, 64, 0, 0, P, P, P, 1, 2, P, big, 0) == 5         # accumulate selector
    assert ex(P, P, P, 256, 512, 512, 64, 0, 0, P, P, P + 4, 1, 0, P, big, 0) == 3     # db alignment
    need0 = raw.mxfp4_linear_backward_ex_workspace(256, 512, 512, 0)
    need1 = raw.mxfp4_linear_backward_ex_workspace(256, 512, 512, 1)
    assert need0 == raw.mxfp4_linear_backward_workspace(256, 512, 512) and need1 > need0 and need1 % 256 == 0
    assert ex(P, P, P, 256, 512, 512, 64, 0, 0, P, P, P, 1, 0, P, need0, 0) == 6       # the bias scratch is missing
    assert raw.mxfp4_linear_backward_ex_workspace(256, 0, 512, 1) == 0
    # fused-producer variant
    gf = raw.mxfp4_gemm_fused
    #      x  rows cols ld  rd g   rnd seed tag Bc Bs N    alpha C  ldc out stream
    assert gf(P, 256, 512, 512, 1, 64, 0, 0, 1, 0, P, 128, 1.0, P, 128, 0, 0) == 1          # B codes NULL
    assert gf(P, 256, 512, 512, 1, 256, 0, 0, 1, P, P, 128, 1.0, P, 128, 0, 0) == 4         # g = 256 is not taken
    assert gf(P, 256, 512, 512, 1, 0, 0, 0, 1, P, P, 128, 1.0, P, 128, 0, 0) == 4           # nor g = 0
    assert gf(P, 256, 384, 384, 1, 64, 0, 0, 1, P, P, 128, 1.0, P, 128, 0, 0) == 2          # K % 256
    assert gf(P, 384, 256, 256, 0, 64, 0, 0, 1, P, P, 128, 1.0, P, 128, 0, 0) == 2          # K = rows for reduce_dim 0
    assert gf(P, 256, 512, 512, 1, 64, 0, 0, 1, P, P, 100, 1.0, P, 128, 0, 0) == 2          # N % 8
    assert gf(P, 256, 512, 512, 1, 64, 0, 0, 1, P, P, 128, 1.0, P, 64, 0, 0) == 2           # ldc < N
    assert gf(P, 256, 512, 512, 1, 64, 5, 0, 1, P, P, 128, 1.0, P, 128, 0, 0) == 5          # rounding
    assert gf(P, 256, 512, 512, 1, 64, 0, 0, 1, P, P + 8, 128, 1.0, P, 128, 0, 0) == 3      # alignment
    lf = raw.mxfp4_linear_backward_fused
    assert lf(P, P, P, 256, 512, 512, 256, 0, 0, P, P, 0, P, big, 0) == 4
    assert lf(P, P, P, 256, 384, 512, 64, 0, 0, P, P, 0, P, big, 0) == 2                    # m % 256
    assert lf(P, P, P, 256, 512, 512, 64, 0, 0, P, P, 0, P, 1024, 0) == 6
    assert lf(P, P, P, 256, 512, 512, 64, 0, 0, 0, P, 0, P, big, 0) == 1
    # split form
    qo = raw.mxfp4_quantize_operands
    assert qo(P, P, 0, 256, 512, 512, 64, 0, 0, P, big, 0) == 1
    assert qo(P, P, P, 256, 500, 512, 64, 0, 0, P, big, 0) == 2
    assert qo(P, P, P, 256, 512, 512, 96, 0, 0, P, big, 0) == 4
    assert qo(P, P, P, 256, 512, 512, 64, 9, 0, P, big, 0) == 5
    assert qo(P, P, P, 256, 512, 512, 64, 0, 0, P, 1024, 0) == 6
    off = (C.c_size_t * 8)()
    raw.mxfp4_operand_layout(256, 512, 512, off)
    assert list(off) == sorted(off) and off[0] == 0 and all(o % 1024 == 0 for o in off)
    assert off[7] + lib.mxfp4_scale_bytes(512, 256) <= raw.mxfp4_linear_backward_workspace(256, 512, 512)
    assert off[1] - off[0] >= 256 * 512 // 2 and off[2] - off[1] >= lib.mxfp4_scale_bytes(256, 512)
    # quantiser with a given transform matrix
    tq = raw.mxfp4_transform_quantize
    #      x  rows cols ld  rd g   T  rnd seed tag codes scales layout y stream
    assert tq(P, 128, 256, 256, 1, 64, 0, 0, 0, 1, P, P, 1, 0, 0) == 1            # T NULL
    assert tq(P, 128, 256, 256, 1, 64, P, 0, 0, 1, 0, P, 1, 0, 0) == 1            # neither codes nor y
    assert tq(P, 128, 256, 256, 1, 256, P, 0, 0, 1, P, P, 1, 0, 0) == 4           # g = 256 not taken
    assert tq(P, 128, 256, 256, 1, 0, P, 0, 0, 1, P, P, 1, 0, 0) == 4
    assert tq(P, 128, 256, 256, 1, 64, P + 2, 0, 0, 1, P, P, 1, 0, 0) == 3        # T alignment
    assert tq(P, 128, 256, 256, 1, 64, P, 4, 0, 1, P, P, 1, 0, 0) == 5            # rounding
    assert tq(P, 128, 250, 256, 1, 64, P, 0, 0, 1, P, P, 1, 0, 0) == 2            # K % 32
    # measurement aid
    assert raw.mxfp4_fp4_ceiling(0, C.byref(C.c_int64(0)), 0) == 2
    assert raw.mxfp4_fp4_ceiling(64, None, 0) == 2
    assert raw.mxfp4_fp4_ceiling(20000001, C.byref(C.c_int64(0)), 0) == 2      # beyond the documented cap (about two seconds of device time)


def test_binding_fails_loudly_without_library(tmp_path, monkeypatch):
    """The product path has no CPU fallback: a missing shared library is an ImportError."""
    import importlib.util
    src = os.path.join(ROOT, "paper_2502_20586_b200", "binding.py")
    dst = tmp_path / "binding_copy.py"
    dst.write_text(open(src).read())
    spec = importlib.util.spec_from_file_location("binding_copy", dst)
    mod = importlib.util.module_from_spec(spec)
    with pytest.raises(ImportError):
        spec.loader.exec_module(mod)


def test_header_is_plain_c(tmp_path):
    """The boundary is a C ABI: include/mxfp4.h compiles as C99 and as C++ with nothing but the standard headers."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no gcc")
    src = tmp_path / "use_header.c"
    src.write_text('#include "include/mxfp4.h"\nint main(void) { return (int)MXFP4_ROUND_SR16 + (int)MXFP4_ERR_TIMEOUT; }\n')
    for cmd in (["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror"], ["g++", "-std=c++11", "-Wall", "-Wextra", "-Werror", "-x", "c++"]):
        subprocess.run(cmd + ["-I", ROOT, "-fsyntax-only", str(src)], check=True)


def test_extension_calls_reject_bad_arguments_before_touching_the_device():
    """FP8 forward and MXINT4 entry points: the same error discipline as the main calls (no GPU needed)."""
    from paper_2502_20586_b200 import binding as mx
    raw = mx.lib()
    P = 4096                                                        # any 16-byte aligned non-null address: never dereferenced
    assert raw.mxfp4_fp8_quantize(None, 8, 64, 64, P, P, 0) == 1
    assert raw.mxfp4_fp8_quantize(P, 8, 60, 64, P, P, 0) == 2       # cols % 8
    assert raw.mxfp4_fp8_quantize(P, 8, 64, 64, P, P + 4, 0) == 3   # the scale pair must be 8-byte aligned
    assert raw.mxfp4_fp8_gemm(P, None, P, P, 128, 8, 128, P, 8, 0, 0) == 1
    assert raw.mxfp4_fp8_gemm(P, P, P, P, 128, 8, 96, P, 8, 0, 0) == 2      # K % 128
    assert raw.mxfp4_fp8_gemm(P, P, P, P, 128, 8, 128, P, 8, 7, 0) == 5
    assert raw.mxfp4_linear_forward_fp8_workspace(0, 1, 1) == 0
    need = raw.mxfp4_linear_forward_fp8_workspace(256, 512, 384)
    assert need >= 256 * 512 + 384 * 512 + 16
    assert raw.mxfp4_linear_forward_fp8(P, P, 256, 512, 384, P, 0, P, need - 1, 0) == 6
    assert raw.mxfp4_linear_forward_fp8(P, P, 256, 500, 384, P, 0, P, need, 0) == 2
    assert raw.mxfp4_int4_quantize(P, 128, 256, 256, 1, 64, 2, 0, 0, P, P, P, 0) == 5      # the 16-bit dither is an MXFP4 mode
    assert raw.mxfp4_int4_quantize(P, 128, 256, 256, 1, 48, 0, 0, 0, P, P, P, 0) == 4
    assert raw.mxfp4_int4_quantize(P, 128, 256, 256, 1, 64, 0, 0, 0, P, P, None, 0) == 1
    assert raw.mxfp4_int4_gemm(P, None, P, P, 128, 8, 128, 1.0, P, 8, 0, 0) == 1
    assert raw.mxfp4_int4_gemm(P, P, P, P, 128, 12, 128, 1.0, P, 12, 0, 0) == 2
