// Element-wise kernels of the two extensions of the recipe (the GEMMs are in gemm_f8.cu):
//   - per-tensor E4M3 quantisation for the FP8 forward pass (Section 4.1; supplementary FP8 results);
//   - MXINT4 elements (Section 3, opening remark): Algorithm 1 / 2 with 4-bit integers in place of E2M1.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.h"
#include "quant_math.cuh"

namespace mx {
namespace {

// ---------------------------------------------------------------- FP8 forward: one scale per tensor
// Pass 1: amax of |x| as the bit pattern of a non-negative float (bf16 magnitudes order like their 15-bit patterns);
// the maximum over the grid is order-independent, so the result is reproducible.
__global__ void fp8_amax_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, uint32_t* amax_bits) {
    const int64_t vec_per_row = cols >> 3, total = rows * vec_per_row;
    uint32_t m = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / vec_per_row, c = (i - r * vec_per_row) << 3;
        const uint4 v = *reinterpret_cast<const uint4*>(x + r * ld + c);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) m = max(m, max(w[j] & 0x7FFFu, (w[j] >> 16) & 0x7FFFu));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((threadIdx.x & 31) == 0 && m != 0) atomicMax(amax_bits, m << 16);
}

// cvt.rn.satfinite.e4m3x2.f32: two floats -> two E4M3 bytes (`lo` in the low byte); nearest-even, saturating at 448.
__device__ __forceinline__ uint32_t cvt_e4m3x2_rn(float lo, float hi) {
    uint16_t d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}

// Pass 2: scale = 448 / amax in fp32 (1 for an all-zero tensor); code = E4M3(fp32(x * scale)).
__global__ void fp8_quantize_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, float* scale_io,
                                    uint8_t* __restrict__ codes) {
    const float amax = scale_io[1];
    const float sf = amax > 0.0f ? 448.0f / amax : 1.0f;
    if (blockIdx.x == 0 && threadIdx.x == 0) scale_io[0] = sf;
    const int64_t vec_per_row = cols >> 3, total = rows * vec_per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / vec_per_row, c = (i - r * vec_per_row) << 3;
        const uint4 v = *reinterpret_cast<const uint4*>(x + r * ld + c);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t out[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const float a0 = __fmul_rn(__uint_as_float(w[2 * j] << 16), sf), a1 = __fmul_rn(__uint_as_float(w[2 * j] & 0xFFFF0000u), sf);
            const float a2 = __fmul_rn(__uint_as_float(w[2 * j + 1] << 16), sf), a3 = __fmul_rn(__uint_as_float(w[2 * j + 1] & 0xFFFF0000u), sf);
            out[j] = cvt_e4m3x2_rn(a0, a1) | (cvt_e4m3x2_rn(a2, a3) << 16);
        }
        *reinterpret_cast<uint2*>(codes + r * cols + c) = make_uint2(out[0], out[1]);
    }
}

// ---------------------------------------------------------------- MXINT4: integers -7..7 with one E8M0 scale per 32
// E4M3 byte that holds the integer q in [0, 7] exactly (the tensor core reads the elements as E4M3).
__device__ __forceinline__ uint32_t e4m3_of_small_int(uint32_t q) {
    // 0, 1 = 1.0 2^0, 2, 3 = 1.5 2^1, 4, 5 = 1.25 2^2, 6 = 1.5 2^2, 7 = 1.75 2^2   (bias 7, three mantissa bits)
    return (0x4E4C4A4844403800ull >> (8 * q)) & 0xFFu;
}

// One thread per MX block of 32 fp32 values.  Scale: the rule of Algorithms 1 / 2 with emax_elem = 2 (largest power of
// two among the elements is 4).  SR (Algorithm 2): w = (3/4) |v| / X < 6, rounded on the integer grid with the dither
// of Eq. 1-2 discretised to the element's 8-bit draw r: up iff 256 frac >= r + 1/2.  Exactly: u = floor(512 w) =
// floor(3 * (128 |v| / X)), where 128 |v| / X is an exact power-of-two scaling and the product by 3 is rounded toward
// zero (floor of a toward-zero rounding of a non-negative real equals the floor of the real); then q = u >> 9 and
// up iff (u & 511) >= 2 r + 1.  RN (Algorithm 1): nearest integer, ties to even, saturating at 7.
__global__ void mxint4_quantize_kernel(const float* __restrict__ y, int64_t R, int64_t K, int rounding, uint64_t seed, uint32_t stream_tag,
                                       uint8_t* __restrict__ codes, uint8_t* __restrict__ scales) {
    const int64_t nkb = K >> 5, blk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (blk >= R * nkb) return;
    const int64_t r = blk / nkb, kb = blk - r * nkb;
    float v[32];
    const float4* src = reinterpret_cast<const float4*>(y + r * K + kb * 32);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float4 f = src[i];
        v[4 * i] = f.x; v[4 * i + 1] = f.y; v[4 * i + 2] = f.z; v[4 * i + 3] = f.w;
    }
    float amax = 0.0f;
#pragma unroll
    for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(v[i]));
    const uint32_t byte = e8m0_from_amax(amax);
    scales[sf_native_offset(r, kb, (nkb + 3) >> 2)] = (uint8_t)byte;
    uint32_t out[8];
    if (byte == 255u) {
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = 0u;
    } else {
        const int e = (int)byte - 127;
        uint32_t rw[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u};
        if (rounding == 0) sr_draws32(seed, stream_tag, (uint64_t)(r * K + kb * 32), rw);
        const int sh = (rounding == 0 ? 7 : 0) - e;                      // |v| 2^sh, in two exact steps
        const float p1 = pow2f_wide(sh / 2), p2 = pow2f_wide(sh - sh / 2);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float a = fabsf(v[i]) * p1 * p2;
            uint32_t q;
            if (rounding == 0) {
                const uint32_t u = (uint32_t)__fmul_rz(a, 3.0f);         // floor(512 w), w < 6
                const uint32_t rr = (rw[i >> 2] >> (8 * (i & 3))) & 0xFFu;
                q = (u >> 9) + ((u & 511u) >= 2u * rr + 1u ? 1u : 0u);
            } else {
                q = (uint32_t)fminf(rintf(a), 7.0f);
            }
            const uint32_t code = e4m3_of_small_int(q) | ((__float_as_uint(v[i]) >> 24) & 0x80u);
            if ((i & 3) == 0) out[i >> 2] = code; else out[i >> 2] |= code << (8 * (i & 3));
        }
    }
    uint4* dst = reinterpret_cast<uint4*>(codes + r * K + kb * 32);
    dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
    dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
}

}  // namespace

cudaError_t launch_fp8_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, float* scale, cudaStream_t stream) {
    cudaError_t e = cudaMemsetAsync(scale + 1, 0, sizeof(float), stream);
    if (e != cudaSuccess) return e;
    const int64_t vecs = rows * (cols >> 3);
    const unsigned grid = (unsigned)(vecs / 256 + 1 < 148 * 16 ? vecs / 256 + 1 : 148 * 16);
    fp8_amax_kernel<<<grid, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(x), rows, cols, ld, reinterpret_cast<uint32_t*>(scale + 1));
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    fp8_quantize_kernel<<<grid, 256, 0, stream>>>(static_cast<const __nv_bfloat16*>(x), rows, cols, ld, scale, codes);
    return cudaGetLastError();
}

cudaError_t launch_mxint4_quantize(const float* y, int64_t R, int64_t K, int rounding, uint64_t seed, uint32_t stream_tag,
                                   uint8_t* codes, uint8_t* scales, cudaStream_t stream) {
    const int64_t blocks = R * (K >> 5);
    mxint4_quantize_kernel<<<(unsigned)((blocks + 127) / 128), 128, 0, stream>>>(y, R, K, rounding, seed, stream_tag, codes, scales);
    return cudaGetLastError();
}

}  // namespace mx
