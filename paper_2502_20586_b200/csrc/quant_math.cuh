// Per-element arithmetic of the quantiser: Philox4x32-10, the sign vector, the in-register Hadamard
// butterflies, the E8M0 scale rule and the E2M1 encoders (Algorithms 1 and 2).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace mx {

// ---------------------------------------------------------------- Philox4x32-10 (counter-based)
// key = (seed lo, seed hi); counter = (index lo, index hi, stream_tag, domain).
// domain 0: sign vector (stream_tag 0, index = j / 128).  domain 1: SR draws (index = element / 16).
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int i = 0; i < 10; ++i) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint32_t u4_word(const uint4& v, int i) {
    return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w;
}

// The 32 sign bits of elements [32 w, 32 w + 32) of the g-long sign vector (bit set = -1).
__device__ __forceinline__ uint32_t sign_word(uint64_t seed, int w) {
    const uint4 o = philox4x32_10((uint32_t)(w >> 2), 0u, 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
    return u4_word(o, w & 3);
}

// The 32 8-bit SR draws of elements [i0, i0 + 32), i0 a multiple of 32: two Philox calls, eight words.
__device__ __forceinline__ void sr_draws32(uint64_t seed, uint32_t stream_tag, uint64_t i0, uint32_t (&rw)[8]) {
    const uint64_t idx = i0 >> 4;
    const uint4 a = philox4x32_10((uint32_t)idx, (uint32_t)(idx >> 32), stream_tag, 1u, (uint32_t)seed, (uint32_t)(seed >> 32));
    const uint4 b = philox4x32_10((uint32_t)(idx + 1), (uint32_t)((idx + 1) >> 32), stream_tag, 1u, (uint32_t)seed, (uint32_t)(seed >> 32));
    rw[0] = a.x; rw[1] = a.y; rw[2] = a.z; rw[3] = a.w;
    rw[4] = b.x; rw[5] = b.y; rw[6] = b.z; rw[7] = b.w;
}

// ---------------------------------------------------------------- Hadamard butterflies (Eq. 4)
// In-place Sylvester transform over the 32 values of one thread (natural order, un-normalised).
__device__ __forceinline__ void fwht32(float (&v)[32]) {
#pragma unroll
    for (int h = 1; h < 32; h <<= 1) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            if ((i & h) == 0) {
                const float a = v[i], b = v[i + h];
                v[i] = a + b;
                v[i + h] = a - b;
            }
        }
    }
}
// One butterfly stage across lanes that differ in `lane_mask` (lane bit clear holds the "upper" half).
__device__ __forceinline__ void fwht_cross(float (&v)[32], int lane_mask, int lane) {
    const bool upper = (lane & lane_mask) != 0;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        const float p = __shfl_xor_sync(0xffffffffu, v[i], lane_mask);
        v[i] = upper ? (p - v[i]) : (v[i] + p);
    }
}

__device__ __forceinline__ float inv_sqrt_g(int g) {
    return g == 32 ? 0.17677669529663687f : g == 64 ? 0.125f : g == 128 ? 0.08838834764831845f : g == 256 ? 0.0625f : 1.0f;
}

// ---------------------------------------------------------------- scale rule and encoders
// 2^k as fp32 for k in [-149, 127] (subnormal results included).
__device__ __forceinline__ float pow2f_wide(int k) {
    return k >= -126 ? __uint_as_float((uint32_t)(k + 127) << 23) : __uint_as_float(1u << (k + 149));
}

// Algorithm 1/2 lines 1-2 for MXFP4: shared_exp = floor(log2 amax) - 2 clamped to [-127, 127];
// E8M0 byte = shared_exp + 127 = max(biased exponent of amax - 2, 0); 255 when amax is not finite.
__device__ __forceinline__ uint32_t e8m0_from_amax(float amax) {
    const uint32_t ef = __float_as_uint(amax) >> 23;          // amax >= 0
    return ef == 255u ? 255u : (ef > 2u ? ef - 2u : 0u);
}

// cvt.rn.satfinite.e2m1x2.f32: two floats -> one byte, `lo` in the low nibble; nearest-even, saturating at 6.
__device__ __forceinline__ uint32_t cvt_e2m1x2_rn(float lo, float hi) {
    uint16_t out;
    asm("{\n\t.reg .b8 b;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b, %1, %2;\n\t"
        "cvt.u16.u8 %0, b;\n\t}"
        : "=h"(out) : "f"(hi), "f"(lo));
    return out;
}

// Quantise 32 consecutive fp32 values (one MX block) to 16 bytes of packed E2M1 codes + one E8M0 byte.
//   SR (Algorithm 2): round up iff r + 1/2 < 256 frac, decided on the exact real w = (3/4) y / X.
//     |y| * (3/4 * 2^(-e-126)) is formed with round-up; since every threshold is representable this keeps
//     the decision exact.  The factor 2^-126 places E2M1's subnormal/normal boundary (1.0) on fp32's, so
//     bits(a) >> 22 IS the E2M1 magnitude code of the lower neighbour and the low 22 bits are frac 2^22;
//     adding ((255 - r) << 14 | 0x1fff) carries into bit 22 exactly when r + 1/2 < 256 frac.
//   RN (Algorithm 1): hardware nearest-even convert of y / X.
__device__ __forceinline__ void quantize_block32(const float (&y)[32], int rounding, uint64_t seed, uint32_t stream_tag,
                                                 uint64_t i0, uint32_t (&packed)[4], uint32_t& scale_byte) {
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(y[i]));
    // fmaxf drops NaNs: detect non-finite inputs through the sum of exponents instead
    bool finite = true;
#pragma unroll
    for (int i = 0; i < 32; ++i) finite = finite && ((__float_as_uint(y[i]) & 0x7F800000u) != 0x7F800000u);
    scale_byte = finite ? e8m0_from_amax(amax) : 255u;
    if (scale_byte == 255u) {
        packed[0] = packed[1] = packed[2] = packed[3] = 0u;
        return;
    }
    const int e = (int)scale_byte - 127;
    if (rounding == 0) {
        uint32_t rw[8];
        sr_draws32(seed, stream_tag, i0, rw);
        const bool fast = e <= 21;                                   // 3/4 * 2^(-e-126) representable
        const float c_fast = fast ? 1.5f * pow2f_wide(-e - 127) : 0.0f;
        const int h1 = (-e) / 2, h2 = -e - h1;                       // slow path: exact 2^-e in two steps
        const float p1 = pow2f_wide(h1), p2 = pow2f_wide(h2);
        const float c_slow = __uint_as_float(0x00600000u);           // 3/4 * 2^-126
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t word = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = 8 * q + j;
                const float ay = fabsf(y[i]);
                const float a = fast ? __fmul_ru(ay, c_fast) : __fmul_ru(ay * p1 * p2, c_slow);
                const uint32_t r = (rw[i >> 2] >> (8 * (i & 3))) & 0xFFu;
                const uint32_t t = __float_as_uint(a) + (((r ^ 0xFFu) << 14) | 0x1FFFu);
                const uint32_t code = (t >> 22) | ((__float_as_uint(y[i]) >> 28) & 8u);
                word |= code << (4 * j);
            }
            packed[q] = word;
        }
    } else {
        const float inv_x = pow2f_wide(-e);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t word = 0u;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = 8 * q + 2 * j;
                word |= cvt_e2m1x2_rn(y[i] * inv_x, y[i + 1] * inv_x) << (8 * j);
            }
            packed[q] = word;
        }
    }
}

// Byte offset of the scale of (row r, 32-block k) in the tcgen05 scale-factor tiling: 128-row x 4-block
// tiles of 512 bytes, tile (r/128, k/4) at ((r/128) * n_ktiles + k/4) * 512, inside a tile
// (r % 32) * 16 + ((r % 128) / 32) * 4 + k % 4.
__device__ __forceinline__ int64_t sf_native_offset(int64_t r, int64_t k, int64_t n_ktiles) {
    return ((r >> 7) * n_ktiles + (k >> 2)) * 512 + (r & 31) * 16 + ((r & 127) >> 5) * 4 + (k & 3);
}

}  // namespace mx
