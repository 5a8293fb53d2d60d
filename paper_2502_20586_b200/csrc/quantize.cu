// Blockwise RHT + MXFP4 quantiser kernels (Algorithm 3 lines 3-6, then Algorithm 2 or 1).
//
// Two access patterns:
//   rowwise   - the reduction dimension is the contiguous one (dY for dgrad);
//   transpose - the reduction dimension is the row index of a row-major tensor (W, dY^T, X^T): the tile is
//               staged in shared memory and each thread walks down a column, so the transposition costs no
//               extra pass over HBM.
// In both, one thread owns one MX block (32 consecutive reduce-dim values): the first five butterfly stages,
// the amax, the scale and the 16 bytes of codes need no communication; g > 32 adds log2(g/32) shuffle stages.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.h"
#include "quant_math.cuh"

namespace mx {

__device__ __forceinline__ void unpack_bf16x8(const uint4& q, float* v) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

// v <- v diag(S) H_g / sqrt(g) for the 32 values of this thread; lanes [lane & ~(G/32-1) ...) share a chunk.
template <int G>
__device__ __forceinline__ void rht_in_place(float (&v)[32], uint32_t sign_bits, int lane, int lane_stride) {
    if constexpr (G != 0) {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = (sign_bits >> i) & 1u ? -v[i] : v[i];
        fwht32(v);
        if (G >= 64) fwht_cross(v, lane_stride, lane);
        if (G >= 128) fwht_cross(v, lane_stride * 2, lane);
        if (G >= 256) fwht_cross(v, lane_stride * 4, lane);
        const float c = inv_sqrt_g(G);
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] *= c;
    }
}

// ------------------------------------------------------------------------------------------------ rowwise
// Thread t of the grid owns MX block B = t: row B / (cols/32), columns [32 (B % (cols/32)), +32).
template <int G, bool DUMP_Y>
__global__ void __launch_bounds__(256) quantize_rowwise_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols,
                                                               int64_t ld, int rounding, uint64_t seed, uint32_t stream_tag,
                                                               uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                                                               int sf_native, float* __restrict__ y_out) {
    const int64_t nkb = cols >> 5;
    const int64_t B = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool valid = B < rows * nkb;
    const int64_t row = valid ? B / nkb : 0;
    const int64_t kb = valid ? B - row * nkb : 0;
    const int lane = threadIdx.x & 31;

    float v[32];
    if (valid) {
        const uint4* src = reinterpret_cast<const uint4*>(x + row * ld + kb * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack_bf16x8(__ldg(src + i), v + 8 * i);
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = 0.0f;
    }
    if (G != 0) {
        const uint32_t sb = sign_word(seed, (int)(kb & (G / 32 - 1)));
        rht_in_place<G>(v, sb, lane, 1);
    }
    if (!valid) return;
    if (DUMP_Y) {
        float4* dst = reinterpret_cast<float4*>(y_out + B * 32);
#pragma unroll
        for (int i = 0; i < 8; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        return;
    }
    uint32_t packed[4], sbyte;
    quantize_block32(v, rounding, seed, stream_tag, (uint64_t)B * 32u, packed, sbyte);
    reinterpret_cast<uint4*>(codes)[B] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
    const int64_t so = sf_native ? sf_native_offset(row, kb, (nkb + 3) >> 2) : B;
    scales[so] = (uint8_t)sbyte;
}

// ---------------------------------------------------------------------------------------------- transpose
// CTA tile: 256 rows (reduce dim) x 64 columns, 256 threads.  Warp w owns columns [8w, 8w+8); lane = 4*rg + cp
// owns rows [32 rg, 32 rg + 32) of the column pair cp.  Shared memory holds the tile as 32-bit words
// (two bf16 columns each), 32 words per row, each row rotated by 4*(row/32) words: the 16-byte tile loads
// and the column walks are both bank-conflict free.
constexpr int kTrRows = 256;
constexpr int kTrCols = 64;

template <int G, bool DUMP_Y>
__global__ void __launch_bounds__(256) quantize_transpose_kernel(const __nv_bfloat16* __restrict__ x, int64_t rows, int64_t cols,
                                                                 int64_t ld, int rounding, uint64_t seed, uint32_t stream_tag,
                                                                 uint8_t* __restrict__ codes, uint8_t* __restrict__ scales,
                                                                 int sf_native, float* __restrict__ y_out) {
    __shared__ __align__(16) uint32_t tile[kTrRows * 32];
    const int tid = threadIdx.x;
    const int64_t col0 = (int64_t)blockIdx.x * kTrCols;
    const int64_t row0 = (int64_t)blockIdx.y * kTrRows;

    // stage: thread t loads 16-byte chunk (t % 8) of rows t/8 + 32 i
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = (tid >> 3) + 32 * i;
        const int c = tid & 7;
        uint4 q = make_uint4(0u, 0u, 0u, 0u);
        if (row0 + r < rows && col0 + c * 8 < cols)
            q = __ldg(reinterpret_cast<const uint4*>(x + (row0 + r) * ld + col0 + c * 8));
        const int rot = (c + (r >> 5)) & 7;
        *reinterpret_cast<uint4*>(&tile[r * 32 + rot * 4]) = q;
    }
    __syncthreads();

    const int warp = tid >> 5, lane = tid & 31;
    const int rg = lane >> 2, cp = lane & 3;
    const int wcol = warp * 4 + cp;                       // word column inside the tile
    float v0[32], v1[32];                                 // the two columns of the pair
#pragma unroll
    for (int r = 0; r < 32; ++r) {
        const uint32_t w = tile[(rg * 32 + r) * 32 + ((wcol + 4 * rg) & 31)];
        v0[r] = __uint_as_float(w << 16);
        v1[r] = __uint_as_float(w & 0xFFFF0000u);
    }
    const int64_t krow = row0 + rg * 32;                  // first reduce-dim index of this thread's block
    if (G != 0) {
        const uint32_t sb = sign_word(seed, (int)((krow >> 5) & (G / 32 - 1)));
        rht_in_place<G>(v0, sb, lane, 4);
        rht_in_place<G>(v1, sb, lane, 4);
    }
    if (krow >= rows) return;
    const int64_t nkb = rows >> 5;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int64_t col = col0 + 2 * wcol + h;          // output row
        if (col >= cols) continue;
        float(&v)[32] = h == 0 ? v0 : v1;
        if (DUMP_Y) {
            float4* dst = reinterpret_cast<float4*>(y_out + col * rows + krow);
#pragma unroll
            for (int i = 0; i < 8; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            continue;
        }
        uint32_t packed[4], sbyte;
        quantize_block32(v, rounding, seed, stream_tag, (uint64_t)(col * rows + krow), packed, sbyte);
        *reinterpret_cast<uint4*>(codes + col * (rows >> 1) + (krow >> 1)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        const int64_t kb = krow >> 5;
        const int64_t so = sf_native ? sf_native_offset(col, kb, (nkb + 3) >> 2) : col * nkb + kb;
        scales[so] = (uint8_t)sbyte;
    }
}

// ---------------------------------------------------------------------------------------------- launchers
template <bool DUMP_Y>
static cudaError_t launch(const QuantArgs& a, cudaStream_t stream) {
    if (quant_tc_eligible(a)) return launch_quantize_tc(a, DUMP_Y, stream);
    const __nv_bfloat16* x = static_cast<const __nv_bfloat16*>(a.x);
    if (a.reduce_dim == 1) {
        const int64_t nblocks = a.rows * (a.cols / 32);
        const unsigned grid = (unsigned)((nblocks + 255) / 256);
#define MX_ROW(G_)                                                                                            \
    quantize_rowwise_kernel<G_, DUMP_Y><<<grid, 256, 0, stream>>>(x, a.rows, a.cols, a.ld, a.rounding, a.seed, \
                                                                   a.stream_tag, a.codes, a.scales, a.sf_native, a.y_out)
        switch (a.g) {
            case 0: MX_ROW(0); break;
            case 32: MX_ROW(32); break;
            case 64: MX_ROW(64); break;
            case 128: MX_ROW(128); break;
            case 256: MX_ROW(256); break;
            default: return cudaErrorInvalidValue;
        }
#undef MX_ROW
    } else {
        const dim3 grid((unsigned)((a.cols + kTrCols - 1) / kTrCols), (unsigned)((a.rows + kTrRows - 1) / kTrRows));
#define MX_TR(G_)                                                                                               \
    quantize_transpose_kernel<G_, DUMP_Y><<<grid, 256, 0, stream>>>(x, a.rows, a.cols, a.ld, a.rounding, a.seed, \
                                                                     a.stream_tag, a.codes, a.scales, a.sf_native, a.y_out)
        switch (a.g) {
            case 0: MX_TR(0); break;
            case 32: MX_TR(32); break;
            case 64: MX_TR(64); break;
            case 128: MX_TR(128); break;
            case 256: MX_TR(256); break;
            default: return cudaErrorInvalidValue;
        }
#undef MX_TR
    }
    return cudaGetLastError();
}

cudaError_t launch_quantize(const QuantArgs& a, cudaStream_t stream) { return launch<false>(a, stream); }
cudaError_t launch_rht_dump(const QuantArgs& a, cudaStream_t stream) { return launch<true>(a, stream); }

}  // namespace mx
