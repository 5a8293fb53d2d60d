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
