// GEMMs on 8-bit element containers (tcgen05 kind::f8f6f4 and kind::mxf8f6f4), for the two extensions of the recipe:
//   plain   C[M, N] = sum_k A[i, k] B[j, k] / (scale_a scale_b),  A, B = E4M3 with one fp32 scale per tensor: the FP8
//           forward pass that the MXFP4 backward is compatible with (Section 4.1; supplementary FP8 results);
//   scaled  C[M, N] = alpha sum_k A[i, k] X_A[i, k / 32] B[j, k] X_B[j, k / 32], E4M3 containers holding the integers
//           -7..7 of MXINT4 elements, one UE8M0 scale per 32 elements along K (scale_vec::1X): the remark that the
//           analysis carries over to MXINT4 (Section 3, opening).
// Structure as the 1-CTA MXFP4 kernel (gemm.cu): persistent, one CTA per SM, 128 x 256 output tile, 4 stages of
// 128 bytes of K (128 elements = four K = 32 MMAs), TMA with 128-byte swizzle, fp32 accumulator in TMEM; scales
// (scaled build) travel global -> shared (bulk copy) -> registers -> TMEM (tcgen05.st) through four mover warps.
// Every mbarrier wait is bounded; on expiry the CTA records a status word and unwinds.
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx.cuh"

namespace mx {
namespace {

constexpr int FM = 128, FN = 256;
constexpr int kStagesF = 4;
constexpr uint32_t kABytesF = FM * 128;                       // 16 KB: 128 rows x 128 elements
constexpr uint32_t kBBytesF = FN * 128;                       // 32 KB
constexpr uint32_t kSfTileF = 512;                            // scale tile: 128 rows x 4 K-blocks = one stage of K
constexpr uint32_t kStageBytesF = 50 * 1024;                  // A, B, SFA tile, two SFB tiles, padded to a multiple of 1 KB
constexpr uint32_t kSmemF = kStagesF * kStageBytesF + 1024 + 256;
constexpr uint32_t kSfColF = 256, kSfSlotColsF = 12;          // per stage: 4 SFA + 8 SFB columns
constexpr int kGroupMF = 16;
constexpr int kThreadsF = 10 * 32;
static_assert(kABytesF + kBBytesF + 3 * kSfTileF <= kStageBytesF, "stage layout");

struct ParamsF {
    const uint8_t* sfa;
    const uint8_t* sfb;
    const float* scale_a;                                     // plain build: per-tensor scales on the device
    const float* scale_b;
    void* C;
    int64_t M, N, K, ldc;
    float alpha;
    int out_fp32;
    int m_tiles, n_tiles;
};

__device__ __forceinline__ void tile_coords_f(int t, int m_tiles, int n_tiles, int& mt, int& nt) {
    const int per_group = kGroupMF * n_tiles;
    const int grp = t / per_group;
    const int first_m = grp * kGroupMF;
    const int gm = min(kGroupMF, m_tiles - first_m);
    const int r = t - grp * per_group;
    mt = first_m + r % gm;
    nt = r / gm;
}

// D[tmem] (+)= A[smem] * B[smem]^T, 8-bit floating-point operands (formats in the instruction descriptor); K = 32.
__device__ __forceinline__ void tc_mma_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Same with one UE8M0 scale per row and 32 elements of K (the MMA's whole K): kind::mxf8f6f4, scale_vec::1X.
__device__ __forceinline__ void tc_mma_mxf8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t sfa_tmem, uint32_t sfb_tmem, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa_tmem), "r"(sfb_tmem)
        : "memory");
}

template <bool SCALED>
__global__ void __launch_bounds__(kThreadsF, 1)
gemm_f8_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const ParamsF p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStagesF * kStageBytesF);
    uint64_t* full_bar = bars;                              // [kStagesF]  TMA -> MMA, scale movers
    uint64_t* empty_bar = full_bar + kStagesF;              // [kStagesF]  MMA -> TMA
    uint64_t* sf_full = empty_bar + kStagesF;               // [kStagesF]  scale movers -> MMA
    uint64_t* tmem_full = sf_full + kStagesF;               // MMA -> epilogue
    uint64_t* tmem_empty = tmem_full + 1;                   // epilogue -> MMA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.m_tiles * p.n_tiles;
    const int num_kt = (int)(p.K >> 7);                       // 128-element pipeline steps = scale tiles along K
    const uint32_t my_tiles = blockIdx.x < (uint32_t)num_tiles ? ((uint32_t)num_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;
    const uint32_t total = my_tiles * (uint32_t)num_kt;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStagesF; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); mbar_init(&sf_full[s], 4); }
        mbar_init(tmem_full, 1);
        mbar_init(tmem_empty, 4);
        *abort_flag = 0;
        mbar_fence_init();
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
                int mt, nt;
                tile_coords_f(t, p.m_tiles, p.n_tiles, mt, nt);
                const int n_row_tiles = min(FN / 128, (int)((p.N - (int64_t)nt * FN + 127) >> 7));
                for (int kt = 0; kt < num_kt; ++kt, ++it) {
                    const int s = it % kStagesF;
                    if (!(ok = mbar_wait(&empty_bar[s], ((it / kStagesF) & 1) ^ 1, abort_flag))) break;
                    uint8_t* st = smem + s * kStageBytesF;
                    mbar_expect_tx(&full_bar[s], kABytesF + kBBytesF + (SCALED ? kSfTileF * (1 + n_row_tiles) : 0u));
                    tma_load_2d(st, &tmap_a, &full_bar[s], kt * 128, mt * FM);
                    tma_load_2d(st + kABytesF, &tmap_b, &full_bar[s], kt * 128, nt * FN);
                    if (SCALED) {
                        bulk_load(st + kABytesF + kBBytesF, p.sfa + ((int64_t)mt * num_kt + kt) * kSfTileF, kSfTileF, &full_bar[s]);
                        for (int j = 0; j < n_row_tiles; ++j)
                            bulk_load(st + kABytesF + kBBytesF + (1 + j) * kSfTileF,
                                      p.sfb + ((int64_t)(nt * (FN / 128) + j) * num_kt + kt) * kSfTileF, kSfTileF, &full_bar[s]);
                    }
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // instruction descriptor: A = B = E4M3 (format 0), K-major, N >> 3 at bit 17, M >> 4 at bit 24;
            // plain: D = fp32 (bits 4-5 = 1); scaled: scale format UE8M0 (bit 23), scale byte ids at bits 4 (B) and 29 (A)
            const uint32_t idesc_base = ((uint32_t)(FN >> 3) << 17) | ((uint32_t)(FM >> 4) << 24) | (SCALED ? (1u << 23) : (1u << 4));
            uint32_t tile_i = 0;
            bool ok = true;
            for (uint32_t it = 0; it < total; ++it) {
                const int kt = (int)(it % (uint32_t)num_kt);
                const int s = it % kStagesF;
                if (kt == 0) {
                    if (!(ok = mbar_wait(tmem_empty, (tile_i & 1) ^ 1, abort_flag))) break;
                }
                if (!(ok = mbar_wait(&full_bar[s], (it / kStagesF) & 1, abort_flag))) break;
                if (SCALED) {
                    if (!(ok = mbar_wait(&sf_full[s], (it / kStagesF) & 1, abort_flag))) break;
                }
                tc_fence_after_sync();
                const uint32_t st = smem_u32(smem + s * kStageBytesF);
                const uint32_t sfa_t = tmem_base + kSfColF + s * kSfSlotColsF, sfb_t = sfa_t + 4;
#pragma unroll
                for (int kb = 0; kb < 4; ++kb) {                       // K = 32 elements = 32 bytes per MMA
                    const uint64_t adesc = make_smem_desc(st + kb * 32, 16, 1024, 2);
                    const uint64_t bdesc = make_smem_desc(st + kABytesF + kb * 32, 16, 1024, 2);
                    if (SCALED) {
                        const uint32_t sf_id = (uint32_t)kb;              // byte of the 32-bit scale column: K-block kb of the stage
                        tc_mma_mxf8(tmem_base, adesc, bdesc, idesc_base | (sf_id << 29) | (sf_id << 4), sfa_t | (sf_id << 30), sfb_t | (sf_id << 30),
                                    (kt | kb) != 0 ? 1u : 0u);
                    } else {
                        tc_mma_f8(tmem_base, adesc, bdesc, idesc_base, (kt | kb) != 0 ? 1u : 0u);
                    }
                }
                tc_commit(&empty_bar[s]);                // frees the stage and (same ring index) its scale slot
                if (kt == num_kt - 1) { tc_commit(tmem_full); ++tile_i; }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp >= 6) {
        // ------------------------------------------------------------------ scale movers (scaled build only)
        // A 512-byte scale tile is the image of 32 TMEM lanes x 4 columns; each warp writes it into its own lane quadrant.
        if (SCALED) {
            const int q = warp & 3;
            const uint32_t lane_base = (uint32_t)(q * 32) << 16;
            bool ok = true;
            for (uint32_t it = 0; it < total; ++it) {
                const int s = it % kStagesF;
                ok = mbar_wait(&full_bar[s], (it / kStagesF) & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after_sync();
                const uint4* sf = reinterpret_cast<const uint4*>(smem + s * kStageBytesF + kABytesF + kBBytesF) + lane;   // 32 uint4 per tile
                const uint32_t sfa_t = tmem_base + lane_base + kSfColF + s * kSfSlotColsF;
                tmem_st_32x32b_x4(sfa_t, sf[0]);
                tmem_st_32x32b_x8(sfa_t + 4, sf[32], sf[64]);          // B rows 0-127 | 128-255 (rows beyond N: stale bytes, never stored)
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sf_full[s]);
            }
            if (!ok && lane == 0) *abort_flag = 1;
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;
        uint32_t tile_i = 0;
        bool ok = true;
        const float alpha = SCALED ? p.alpha : 1.0f / (*p.scale_a * *p.scale_b);
        for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++tile_i) {
            int mt, nt;
            tile_coords_f(t, p.m_tiles, p.n_tiles, mt, nt);
            ok = mbar_wait(tmem_full, tile_i & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const int64_t row = (int64_t)mt * FM + q * 32 + lane;
            const int64_t col0 = (int64_t)nt * FN;
#pragma unroll 1
            for (int c = 0; c < FN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(tmem_base + ((uint32_t)(q * 32) << 16) + c * 32, r);
                tmem_ld_wait();
                const int64_t col = col0 + c * 32;
                if (row < p.M && col < p.N) {
                    const int nvalid = (int)min((int64_t)32, p.N - col);      // multiple of 8
                    if (p.out_fp32) {
                        float* dst = static_cast<float*>(p.C) + row * p.ldc + col;
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            if (4 * v < nvalid)
                                reinterpret_cast<float4*>(dst)[v] = make_float4(__uint_as_float(r[4 * v]) * alpha, __uint_as_float(r[4 * v + 1]) * alpha,
                                                                                __uint_as_float(r[4 * v + 2]) * alpha, __uint_as_float(r[4 * v + 3]) * alpha);
                    } else {
                        __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.C) + row * p.ldc + col;
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            if (8 * v < nvalid) {
                                uint32_t w[4];
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * v + 2 * j]) * alpha,
                                                                                   __uint_as_float(r[8 * v + 2 * j + 1]) * alpha);
                                    w[j] = *reinterpret_cast<const uint32_t*>(&h);
                                }
                                reinterpret_cast<uint4*>(dst)[v] = make_uint4(w[0], w[1], w[2], w[3]);
                            }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(tmem_empty);
        }
        if (!ok && lane == 0) *abort_flag = 1;
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);     // let copies in flight land before the shared memory goes away
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace

cudaError_t fetch_gemm_f8_status(unsigned int* word) { return device_status_fetch(word); }

cudaError_t gemm_f8_init() {
    cudaError_t e = cudaFuncSetAttribute(gemm_f8_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemF);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(gemm_f8_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemF);
}

cudaError_t launch_gemm_f8(const Gemm8Args& a, cudaStream_t stream) {
    ParamsF p;
    p.sfa = a.sfa; p.sfb = a.sfb; p.scale_a = a.scale_a; p.scale_b = a.scale_b; p.C = a.C;
    p.M = a.M; p.N = a.N; p.K = a.K; p.ldc = a.ldc;
    p.alpha = a.alpha; p.out_fp32 = a.out_fp32;
    p.m_tiles = (int)((a.M + FM - 1) / FM);
    p.n_tiles = (int)((a.N + FN - 1) / FN);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int tiles = p.m_tiles * p.n_tiles;
    const int grid = tiles < sms ? tiles : sms;
    if (a.block_scaled) gemm_f8_kernel<true><<<grid, kThreadsF, kSmemF, stream>>>(a.tmap_a, a.tmap_b, p);
    else gemm_f8_kernel<false><<<grid, kThreadsF, kSmemF, stream>>>(a.tmap_a, a.tmap_b, p);
    return cudaGetLastError();
}

}  // namespace mx
