// Bias gradient of the linear layer (problem statement, Section 2: dL/db = 1 dL/dy): column sums of dY [b, m] in
// fp32.  HBM-bound: dY is read once (2 bytes per element).  Two deterministic passes:
//   1. colsum_partial: CTA (column block of 256, row split) sums its rows; thread = 8 consecutive columns (one 16-byte
//      load per row), warp = 256 columns of a row (512 contiguous bytes), the CTA's 8 warps take rows round-robin and
//      combine through shared memory in warp order.  Result: partial[split][m].
//   2. colsum_finish: db[j] = (accumulate ? db[j] : 0) + sum over splits in split order.
#include <cuda_bf16.h>

#include "kernels.h"

namespace mx {
namespace {

constexpr int kColsPerCta = 256, kWarpsB = 8, kThreadsB = kWarpsB * 32;

__global__ void __launch_bounds__(kThreadsB)
colsum_partial(const __nv_bfloat16* __restrict__ dY, int64_t b, int64_t m, int64_t ld, int64_t rows_per_split, float* __restrict__ partial) {
    __shared__ float red[kWarpsB][kColsPerCta];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t col = (int64_t)blockIdx.x * kColsPerCta + lane * 8;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_split, r1 = min(b, r0 + rows_per_split);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (col < m) {                                        // m % 8 == 0: a thread's 8 columns are all inside or all outside
        const __nv_bfloat16* p = dY + col;
#pragma unroll 4
        for (int64_t r = r0 + warp; r < r1; r += kWarpsB) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(p + r * ld));
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[2 * j] += __uint_as_float(w[j] << 16);
                acc[2 * j + 1] += __uint_as_float(w[j] & 0xFFFF0000u);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) red[warp][lane * 8 + j] = acc[j];
    __syncthreads();
    const int64_t c = (int64_t)blockIdx.x * kColsPerCta + threadIdx.x;
    if (c < m) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kWarpsB; ++w) s += red[w][threadIdx.x];
        partial[(int64_t)blockIdx.y * m + c] = s;
    }
}

__global__ void colsum_finish(const float* __restrict__ partial, int64_t m, int splits, int accumulate, float* __restrict__ db) {
    const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= m) return;
    float s = accumulate ? db[c] : 0.f;
    for (int k = 0; k < splits; ++k) s += partial[(int64_t)k * m + c];
    db[c] = s;
}

}  // namespace

int bias_grad_splits(int64_t b, int64_t m) {
    const int64_t col_blocks = (m + kColsPerCta - 1) / kColsPerCta;
    int64_t splits = (4 * 148 + col_blocks - 1) / col_blocks;          // about four CTAs per SM of a B200 (148); a pure
                                                                        // function of the shape, so the workspace query and the launch agree
    const int64_t max_splits = (b + 63) / 64;                           // at least 64 rows per split
    if (splits > max_splits) splits = max_splits;
    if (splits > 64) splits = 64;
    if (splits < 1) splits = 1;
    return (int)splits;
}

// Room for either form of the first pass: the stand-alone kernel's splits, or one partial row per 128-row band of dY
// when the quantiser launch computes the sums on its way.
size_t bias_grad_workspace(int64_t b, int64_t m) {
    const int64_t bands = (b + 127) / 128, splits = bias_grad_splits(b, m);
    return (size_t)(bands > splits ? bands : splits) * (size_t)m * sizeof(float);
}

cudaError_t launch_bias_finish(const float* partial, int64_t m, int bands, int accumulate, float* db, cudaStream_t stream) {
    colsum_finish<<<(unsigned)((m + 255) / 256), 256, 0, stream>>>(partial, m, bands, accumulate, db);
    return cudaGetLastError();
}

cudaError_t launch_bias_grad(const void* dY, int64_t b, int64_t m, int64_t ld, int accumulate, float* db, float* partial, cudaStream_t stream) {
    const int splits = bias_grad_splits(b, m);
    const int64_t rows_per_split = (b + splits - 1) / splits;
    const dim3 grid((unsigned)((m + kColsPerCta - 1) / kColsPerCta), (unsigned)splits);
    colsum_partial<<<grid, kThreadsB, 0, stream>>>(static_cast<const __nv_bfloat16*>(dY), b, m, ld, rows_per_split, partial);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    colsum_finish<<<(unsigned)((m + 255) / 256), 256, 0, stream>>>(partial, m, splits, accumulate, db);
    return cudaGetLastError();
}

}  // namespace mx
