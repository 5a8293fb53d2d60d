// Internal launch interfaces between the C-ABI layer (api.cu) and the kernel files.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mx {

struct QuantArgs {
    const void* x;        // bf16 [rows, cols], leading dimension ld
    int64_t rows, cols, ld;
    int reduce_dim;       // 1: reduce along cols; 0: reduce along rows (transposed output)
    int g;                // 0, 32, 64, 128, 256
    int rounding;         // 0 SR, 1 RN, 2 SR with the 16-bit dither
    uint64_t seed;
    uint32_t stream_tag;
    uint8_t* codes;
    uint8_t* scales;
    int sf_native;
    float* y_out;         // only for the transform dump
    CUtensorMap tmap_x;   // x as [rows, cols] bf16, box 64 cols x 128 rows, 128-byte swizzle (tensor-core path)
    bool has_tmap;
    const void* custom_t = nullptr;   // bf16 [g, g] row-major: transform matrix given by the caller instead of diag(S) H_g / sqrt(g) (tensor-core path, g <= 128)
};

// Tensor-core transform path (quantize_tc.cu): g in {32, 64, 128} and reduce length a multiple of 128.
bool quant_tc_eligible(const QuantArgs& a);
cudaError_t quant_tc_init();
cudaError_t launch_quantize_tc(const QuantArgs& a, bool dump_y, cudaStream_t stream);
// Up to kQuantMaxViews eligible views sharing g, seed, rounding and scale layout, in ONE launch.
constexpr int kQuantMaxViews = 4;
// lite: the small-footprint build (g <= 128) that can share an SM with the small build of the pair GEMM.
// dual: n = 2, a[0] / a[1] = the row-wise and the transposed view of ONE tensor (both extents multiples of 128): every tile of it is read once.
// col_sums (dual only, may be null): fp32 [rows / 128, cols] receives the column sums of every 128-row band of that tensor.
cudaError_t launch_quantize_tc_group(const QuantArgs* a, int n, bool dump_y, cudaStream_t stream, bool lite = false, bool dual = false,
                                     float* col_sums = nullptr);

cudaError_t launch_quantize(const QuantArgs& a, cudaStream_t stream);
cudaError_t launch_rht_dump(const QuantArgs& a, cudaStream_t stream);

struct GemmArgs {
    CUtensorMap tmap_a;   // codes [M, K/2] bytes, box 128 B x 128 rows, 128-byte swizzle
    CUtensorMap tmap_b;   // codes [N, K/2] bytes, box 128 B x BN rows
    CUtensorMap tmap_b_half;   // same tensor, box 128 B x 128 rows (CTA-pair kernel: each CTA loads half a B tile)
    CUtensorMap tmap_c;   // output [M, N] (leading dimension ldc): box 64 bytes x 32 rows, 64-byte swizzle (pair kernel's stores)
    bool has_tmap_c;      // false when C cannot be described by a tensor map: the kernel then stores directly
    bool use_pair;        // run the CTA-pair kernel (gemm_pair.cu)
    bool lite = false;    // pair kernel only: the small-footprint build that leaves room on the SM for a co-resident quantiser
    const uint8_t* sfa;   // native scale layout
    const uint8_t* sfb;
    int64_t M, N, K;
    float alpha;
    void* C;
    int64_t ldc;
    int out_fp32;
    int accumulate;       // C += alpha A B^T instead of C = (fp32 output only)
};

constexpr int kGemmBM = 128;
constexpr int kGemmBN = 256;
constexpr int kGemmBKBytes = 128;   // 256 E2M1 elements per pipeline stage

// Bias gradient: db [m] (fp32) = (accumulate ? db : 0) + column sums of bf16 dY [b, m]; `partial` is scratch of
// bias_grad_workspace(b, m) bytes.
size_t bias_grad_workspace(int64_t b, int64_t m);
cudaError_t launch_bias_grad(const void* dY, int64_t b, int64_t m, int64_t ld, int accumulate, float* db, float* partial, cudaStream_t stream);
// Second pass alone: db [m] = (accumulate ? db : 0) + the `bands` rows of partial [bands, m] added in order (the first pass
// was done by the dual-view quantiser launch, which holds every tile of dY in shared memory anyway).
cudaError_t launch_bias_finish(const float* partial, int64_t m, int bands, int accumulate, float* db, cudaStream_t stream);

// Each kernel file keeps its own device status word (set when a bounded wait expires); these read and clear them.
cudaError_t fetch_gemm_status(unsigned int* word);
cudaError_t fetch_gemm_pair_status(unsigned int* word);
cudaError_t fetch_quant_tc_status(unsigned int* word);
cudaError_t fetch_fp4_ceiling_status(unsigned int* word);

// GEMM with the RHT + quantiser of its A operand fused into the kernel (gemm_fused.cu): A = x or x^T in bf16.
struct FusedGemmArgs {
    CUtensorMap tmap_x;   // x as [rows, cols] bf16, box 64 cols x 128 rows, 128-byte swizzle
    bool has_tmap_x;
    CUtensorMap tmap_b;   // codes [N, K/2] bytes, box 128 B x 128 rows
    const uint8_t* sfb;   // native scale layout
    int64_t M, N, K;
    float alpha;
    void* C;
    int64_t ldc;
    int out_fp32;
    int g;                // 32, 64, 128
    int reduce_dim;       // 1: A = x; 0: A = x^T
    int rounding;
    uint64_t seed;
    uint32_t stream_tag;
};
bool gemm_fused_eligible(const FusedGemmArgs& a);
cudaError_t launch_gemm_fused(const FusedGemmArgs& a, cudaStream_t stream);
cudaError_t gemm_fused_init();
cudaError_t fetch_gemm_fused_status(unsigned int* word);

// GEMM on 8-bit element containers (gemm_f8.cu): E4M3 operands with per-tensor scales (FP8 forward pass), or E4M3
// containers of MXINT4 integers with one UE8M0 scale per 32 elements (native scale layout, K % 128 == 0).
struct Gemm8Args {
    CUtensorMap tmap_a;   // bytes [M, K], box 128 B x 128 rows, 128-byte swizzle
    CUtensorMap tmap_b;   // bytes [N, K], box 128 B x 256 rows
    bool block_scaled;
    const uint8_t* sfa;   // block_scaled: native scale layout
    const uint8_t* sfb;
    const float* scale_a; // plain: device pointers to the per-tensor scales; C = A B^T / (scale_a scale_b)
    const float* scale_b;
    int64_t M, N, K;
    float alpha;          // block_scaled only
    void* C;
    int64_t ldc;
    int out_fp32;
};
cudaError_t launch_gemm_f8(const Gemm8Args& a, cudaStream_t stream);
cudaError_t gemm_f8_init();
cudaError_t fetch_gemm_f8_status(unsigned int* word);

// Element-wise kernels of the extensions (variants.cu).
// Per-tensor E4M3 quantisation: *scale = 448 / amax(x) (1 for an all-zero tensor), codes = E4M3(x * scale).
// `scale` doubles as the amax scratch word while the call runs.
cudaError_t launch_fp8_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, float* scale, cudaStream_t stream);
// MXINT4 from fp32 pre-quantisation values y [R, K]: per 32-block E8M0 scale (Algorithm 1 / 2 rule), elements rounded
// to integers in [-7, 7] (rounding 0: 3/4 pre-scale + stochastic rounding with the path's Philox draws; 1: nearest),
// stored as E4M3 bytes; scales in the native layout.
cudaError_t launch_mxint4_quantize(const float* y, int64_t R, int64_t K, int rounding, uint64_t seed, uint32_t stream_tag,
                                   uint8_t* codes, uint8_t* scales, cudaStream_t stream);

cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t stream);
cudaError_t gemm_init();            // one-time: opt in to large dynamic shared memory
cudaError_t launch_gemm_pair(const GemmArgs& a, cudaStream_t stream);
cudaError_t gemm_pair_init();

}  // namespace mx
