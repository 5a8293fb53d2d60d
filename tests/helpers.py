"""Test-side helpers: layout decoders written independently of both the CUDA path and the oracle."""
import numpy as np


def sf_native_offsets(rows: int, K: int) -> np.ndarray:
    """Byte offset of the scale of (row, 32-block) in the tcgen05 scale-factor tiling, as documented for
    block-scaled GEMM operands: 128-row x 4-block tiles of 512 bytes, K-tiles fastest; inside a tile the
    32 x 16-byte image holds row % 32 down the 16-byte lines, (row % 128) / 32 across 4-byte groups and
    block % 4 inside a group."""
    nkb = K // 32
    n_ktiles = (nkb + 3) // 4
    r = np.arange(rows)[:, None]
    k = np.arange(nkb)[None, :]
    tile = (r // 128) * n_ktiles + (k // 4)
    return tile * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + (k % 4)


def sf_native_to_linear(buf: np.ndarray, rows: int, K: int) -> np.ndarray:
    return buf[sf_native_offsets(rows, K)]


def sf_linear_to_native(scales: np.ndarray, fill: int = 0) -> np.ndarray:
    rows, nkb = scales.shape
    size = ((rows + 127) // 128) * ((nkb + 3) // 4) * 512
    out = np.full(size, fill, np.uint8)
    out[sf_native_offsets(rows, nkb * 32)] = scales
    return out


def unpack_codes(packed: np.ndarray) -> np.ndarray:
    """[R, K/2] bytes -> [R, K] codes, even k in the low nibble."""
    R, half = packed.shape
    out = np.empty((R, 2 * half), np.uint8)
    out[:, 0::2] = packed & 0xF
    out[:, 1::2] = packed >> 4
    return out


E2M1_STEP_INDEX = np.array([0, 1, 2, 3, 4, 5, 6, 7, 0, -1, -2, -3, -4, -5, -6, -7])   # signed position on the grid

E2M1_MAGNITUDE = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])   # Section 2.1 / Table 1


def dequant(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """[R, K] codes (one per byte) and [R, K/32] E8M0 bytes -> fp64 values (-1)^s * magnitude * 2^(byte - 127)."""
    sign = np.where(codes & 8, -1.0, 1.0)
    return sign * E2M1_MAGNITUDE[codes & 7] * np.exp2(scales.astype(np.float64) - 127.0).repeat(32, axis=1)


def compare_quantised_rows(c, s, oc, os_, max_rate=1e-4):
    """Codes / scale bytes of the same operand rows from the CUDA path (c, s) and from the oracle (oc, os_).

    Where the scale bytes agree, at most `max_rate` of the codes may differ, each by one grid step.  A block whose
    amax sits within fp32 rounding of a power of two may get neighbouring scale bytes on the two sides; such blocks
    are not dropped: the bytes must differ by exactly one and every dequantised value must lie within one step of the
    coarser of the two grids (both results are neighbours of the same real on nested grids).
    Returns the fraction of elements that differ in any way (used to bound the effect on a GEMM output)."""
    same_block = s == os_
    same = same_block.repeat(32, axis=1)
    assert (~same_block).mean() <= max_rate
    diff = (c != oc) & same
    assert diff.mean() <= max_rate, diff.mean()
    assert np.all(np.abs(E2M1_STEP_INDEX[c[diff]] - E2M1_STEP_INDEX[oc[diff]]) <= 1)
    if not same_block.all():
        assert np.all(np.abs(s.astype(np.int64) - os_.astype(np.int64))[~same_block] == 1)
        va, vb = dequant(c, s), dequant(oc, os_)
        xc = np.exp2(np.maximum(s, os_).astype(np.float64) - 127.0).repeat(32, axis=1)     # the coarser grid's unit
        mag = np.maximum(np.abs(va), np.abs(vb)) / xc
        step = np.where(mag <= 2.0, 0.5, np.where(mag <= 4.0, 1.0, 2.0)) * xc
        assert np.all(np.abs(va - vb)[~same] <= step[~same])
    return float(((c != oc) | ~same).mean())


def product_tolerance(rate_a: float, rate_b: float, out_bits: int = 24) -> float:
    """Relative Frobenius bound between two MXFP4 products whose operands differ in the given fractions of elements,
    each by at most one grid step: a differing element changes its term by at most about the term's own size, so
    with zero-mean terms the relative change of a sum is about sqrt(rate); 4 is head-room.  Plus the GEMM's own
    1e-5 and the unit roundoff of the output format (2^-8 for bf16's 8 significand bits)."""
    return 4.0 * np.sqrt(rate_a + rate_b) + 1e-5 + (2.0 ** -8 if out_bits == 8 else 0.0)


def band_rows(n_rows: int) -> np.ndarray:
    """One row in every 128-row band, rotating through the band's four 32-row quadrants and through the rows of a
    quadrant: every output tile, both CTAs of a pair and (over four bands) every epilogue warp's quadrant are hit."""
    i = np.arange((n_rows + 127) // 128)
    r = 128 * i + 32 * (i % 4) + (7 * i) % 32
    return r[r < n_rows]


def chunk_cols(n_cols: int, chunk: int = 32) -> np.ndarray:
    """One column in every `chunk`-column group (every 64-byte store box of a bf16 output for chunk = 32)."""
    j = np.arange((n_cols + chunk - 1) // chunk)
    c = chunk * j + (11 * j) % chunk
    return c[c < n_cols]
