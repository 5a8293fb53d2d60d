// MXFP4 GEMM with the blockwise RHT and the quantiser of its A operand fused into the producer side of the kernel
// (Section 3.2 suggests fusing the transform with the GEMM's operand path; Algorithm 3 lines 3/5 + 7/8 in one kernel):
//     C[M, N] = alpha * Q(A blockdiag(S H_g / sqrt(g))) deq(B)^T,     A = x (reduce_dim 1) or x^T (reduce_dim 0), bf16,
// B already quantised (codes + scales in the tcgen05 tiling).  The A codes and scales never go through global memory.
//
// Per CTA: a 128 x 128 output tile, K-steps of 256 elements.  Per K-step two 128 x 128 bf16 tiles of x arrive by TMA,
// each goes through the transform as a kind::f16 MMA into its own TMEM accumulator (as in quantize_tc.cu), one group
// of four warps per accumulator reads it back (a thread owns one row: four MX blocks), rounds it with the same
// Philox draws, keyed on the element index in the full operand, as the stand-alone quantiser (the codes are
// identical to what that kernel would have written, whichever CTA derives them), stores the packed codes into the
// 128-byte-swizzled K-major stage the kind::mxf4 MMA reads, and moves the scale bytes through a 512-byte image in
// shared memory into the TMEM scale columns of all four lane quadrants.  The B side is the 1-CTA GEMM's: TMA for the
// codes, a bulk copy for the scales, tcgen05.st into TMEM.
//
//   warp 0        TMA producer: x tiles (3-deep ring), B code tiles and B scales (2-deep ring)
//   warp 1        MMA issuer: transform MMAs of K-step i, then the four kind::mxf4 MMAs of K-step i - 1
//   warps 2, 3    idle
//   warps 4..7    quantiser group 0: first 128 elements of every K-step; also moves the B scales
//   warps 8..11   quantiser group 1: second 128 elements of every K-step
//   warps 12..15  epilogue: TMEM -> registers -> alpha -> bf16 / fp32 -> global
//
// Every CTA that works on an output tile re-quantises the A panel of that tile, N / 128 times over the whole
// product: the kernel is bound by the quantiser arithmetic, not by the tensor pipe, and is the slower way to run
// Algorithm 3 on this GPU except for narrow N; it exists to measure exactly that.
// Every mbarrier wait is bounded; on expiry the CTA records a status word and unwinds.
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx.cuh"
#include "quant_math.cuh"

namespace mx {
namespace {

constexpr int FM = 128, FN = 128;
constexpr int kXStages = 3;                                 // bf16 x tiles in flight
constexpr int kStagesF = 2;                                 // K-steps of quantised A codes / B codes / scales
constexpr uint32_t kBoxBytesF = 64 * 2 * 128;               // one TMA box of x: 64 bf16 columns x 128 rows
constexpr uint32_t kXTileBytes = 2 * kBoxBytesF;            // 32 KB
constexpr uint32_t kTBytesF = 2 * kBoxBytesF;               // transform matrix, 128 x 128 bf16
constexpr uint32_t kA4Bytes = FM * kGemmBKBytes;            // 16 KB of codes per K-step
constexpr uint32_t kB4Bytes = FN * kGemmBKBytes;            // 16 KB
constexpr uint32_t kSfTileF = 512;                          // scale tile: 128 rows x 4 K-blocks
constexpr uint32_t kSfStageF = 4 * kSfTileF;                // SFA tile 0, 1 | SFB tile 0, 1
constexpr uint32_t kOffT = kXStages * kXTileBytes;
constexpr uint32_t kOffA4 = kOffT + kTBytesF;
constexpr uint32_t kOffB4 = kOffA4 + kStagesF * kA4Bytes;
constexpr uint32_t kOffSf = kOffB4 + kStagesF * kB4Bytes;
constexpr uint32_t kOffBar = kOffSf + kStagesF * kSfStageF;
constexpr uint32_t kSmemF = kOffBar + 256 + 1024 /*alignment slack*/;
static_assert(kSmemF <= 232448, "shared memory budget");
constexpr uint32_t kMainCol = 0;                            // 128 fp32 accumulator columns of the product
constexpr uint32_t kRhtCol = 128;                           // two transform accumulators of 128 columns
constexpr uint32_t kSfColF = 384;                           // kStagesF slots of (8 SFA + 8 SFB) columns
constexpr uint32_t kSfSlotColsF = 16;
constexpr int kGroupMF = 16;
constexpr int kThreadsF = 16 * 32;

struct FParams {
    const uint8_t* sfb;
    void* C;
    int64_t M, N, K, ldc;
    float alpha;
    int out_fp32;
    int m_tiles, n_tiles;
    int g, reduce_dim;
    uint32_t stream_tag;
    uint64_t seed;
    PipeConsts pipe;
    PhiloxKeys keys;
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

template <int ROUNDING>
__global__ void __launch_bounds__(kThreadsF, 1)
gemm_fused_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ FParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* smem_t = smem + kOffT;
    uint8_t* smem_a4 = smem + kOffA4;
    uint8_t* smem_b4 = smem + kOffB4;
    uint8_t* smem_sf = smem + kOffSf;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kOffBar);
    uint64_t* x_full = bars;                                // [kXStages]  TMA -> transform MMA
    uint64_t* x_empty = x_full + kXStages;                  // [kXStages]  transform MMA -> TMA
    uint64_t* acc_full = x_empty + kXStages;                // [2]         transform MMA -> quantiser group h
    uint64_t* acc_empty = acc_full + 2;                     // [2]         quantiser group h -> transform MMA
    uint64_t* grp_bar = acc_empty + 2;                      // [2]         scale image of group h complete (its four warps)
    uint64_t* b_full = grp_bar + 2;                         // [kStagesF]  TMA (B codes, B scales) -> movers, MMA
    uint64_t* a_full = b_full + kStagesF;                   // [kStagesF]  quantiser groups -> MMA (codes in smem, scales in TMEM)
    uint64_t* stage_empty = a_full + kStagesF;              // [kStagesF]  MMA -> TMA, quantiser groups
    uint64_t* tmem_full = stage_empty + kStagesF;           // MMA -> epilogue
    uint64_t* tmem_empty = tmem_full + 1;                   // epilogue -> MMA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.m_tiles * p.n_tiles;
    const int nkc = (int)(p.K >> 7);                          // 128-element scale chunks along K
    const int num_kt = nkc >> 1;                              // 256-element K-steps (K % 256 == 0)
    const uint32_t my_tiles = blockIdx.x < (uint32_t)num_tiles ? ((uint32_t)num_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;
    const uint32_t total = my_tiles * (uint32_t)num_kt;       // K-steps this CTA runs, over all its tiles
    const bool rowwise = p.reduce_dim == 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kXStages; ++s) { mbar_init(&x_full[s], 1); mbar_init(&x_empty[s], 1); }
        for (int h = 0; h < 2; ++h) { mbar_init(&acc_full[h], 1); mbar_init(&acc_empty[h], 4); mbar_init(&grp_bar[h], 4); }
        for (int s = 0; s < kStagesF; ++s) { mbar_init(&b_full[s], 1); mbar_init(&a_full[s], 8); mbar_init(&stage_empty[s], 1); }
        mbar_init(tmem_full, 1);
        mbar_init(tmem_empty, 4);
        *abort_flag = 0;
        mbar_fence_init();
        prefetch_tensormap(&tmap_x);
        prefetch_tensormap(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    {
        // Transform operand in the 128-byte-swizzled K-major layout: entry (n, k) at box (k / 64), row n, chunk ((k % 64) / 8) ^ (n % 8).
        const uint4 o = philox4x32_10(0u, 0u, 0u, 0u, (uint32_t)p.seed, (uint32_t)(p.seed >> 32));
        const uint32_t sign[4] = {o.x, o.y, o.z, o.w};
        for (int task = threadIdx.x; task < 128 * 16; task += kThreadsF) {
            const int n = task >> 4, c = task & 15;
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int k0 = c * 8 + 2 * j;
                w[j] = transform_entry(n, k0, p.g, sign) | (transform_entry(n, k0 + 1, p.g, sign) << 16);
            }
            const uint32_t off = (uint32_t)(c >> 3) * kBoxBytesF + (uint32_t)n * 128u + (uint32_t)(((c & 7) ^ (n & 7)) << 4);
            *reinterpret_cast<uint4*>(smem_t + off) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        fence_proxy_async_smem();
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
                for (int kt = 0; kt < num_kt && ok; ++kt, ++it) {
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t xi = 2 * it + h;
                        const int xs = xi % kXStages;
                        if (!(ok = mbar_wait(&x_empty[xs], ((xi / kXStages) & 1) ^ 1, abort_flag))) break;
                        const int ktile = 2 * kt + h;                        // 128-wide k-tile
                        const int32_t cx = (rowwise ? ktile : mt) * 128, cy = (rowwise ? mt : ktile) * 128;
                        uint8_t* st = smem + xs * kXTileBytes;
                        mbar_expect_tx(&x_full[xs], kXTileBytes);
                        tma_load_2d(st, &tmap_x, &x_full[xs], cx, cy);
                        tma_load_2d(st + kBoxBytesF, &tmap_x, &x_full[xs], cx + 64, cy);
                    }
                    if (!ok) break;
                    const int s = it % kStagesF;
                    if (!(ok = mbar_wait(&stage_empty[s], ((it / kStagesF) & 1) ^ 1, abort_flag))) break;
                    mbar_expect_tx(&b_full[s], kB4Bytes + 2 * kSfTileF);
                    tma_load_2d(smem_b4 + s * kB4Bytes, &tmap_b, &b_full[s], kt * kGemmBKBytes, nt * FN);
                    bulk_load(smem_sf + s * kSfStageF + 2 * kSfTileF, p.sfb + ((int64_t)nt * nkc + 2 * kt) * kSfTileF, 2 * kSfTileF, &b_full[s]);
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // kind::f16: D = fp32, A = B = bf16, A major at bit 15 (1 = MN-major: the transposing view), N >> 3 at bit 17, M >> 4 at bit 24
            const uint32_t idesc_rht = (1u << 4) | (1u << 7) | (1u << 10) | ((rowwise ? 0u : 1u) << 15) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
            // kind::mxf4: A, B = E2M1, scale = UE8M0, K-major
            const uint32_t idesc_main = (1u << 7) | (1u << 10) | ((uint32_t)(FN >> 3) << 17) | (1u << 23) | ((uint32_t)(FM >> 4) << 24);
            const uint32_t t_addr = smem_u32(smem_t);
            bool ok = true;
            auto main_step = [&](uint32_t j) -> bool {             // the four kind::mxf4 MMAs of K-step j
                const int kt = (int)(j % (uint32_t)num_kt);
                const int s = j % kStagesF;
                if (kt == 0 && !mbar_wait(tmem_empty, ((j / (uint32_t)num_kt) & 1) ^ 1, abort_flag)) return false;
                if (!mbar_wait(&a_full[s], (j / kStagesF) & 1, abort_flag)) return false;
                if (!mbar_wait(&b_full[s], (j / kStagesF) & 1, abort_flag)) return false;
                tc_fence_after_sync();
                const uint32_t a_addr = smem_u32(smem_a4 + s * kA4Bytes), b_addr = smem_u32(smem_b4 + s * kB4Bytes);
                const uint32_t sfa_t = tmem_base + kSfColF + s * kSfSlotColsF, sfb_t = sfa_t + 8;
#pragma unroll
                for (int kb = 0; kb < 4; ++kb) {
                    const uint64_t adesc = make_smem_desc(a_addr + kb * 32, 16, 1024, 2);
                    const uint64_t bdesc = make_smem_desc(b_addr + kb * 32, 16, 1024, 2);
                    const uint32_t sf_id = (uint32_t)(kb & 1) * 2u;
                    const uint32_t idesc = idesc_main | (sf_id << 29) | (sf_id << 4);
                    tc_mma_mxf4(tmem_base + kMainCol, adesc, bdesc, idesc, (sfa_t + 4 * (kb >> 1)) | (sf_id << 30),
                                (sfb_t + 4 * (kb >> 1)) | (sf_id << 30), (kt | kb) != 0 ? 1u : 0u);
                }
                tc_commit(&stage_empty[s]);
                if (kt == num_kt - 1) tc_commit(tmem_full);
                return true;
            };
            for (uint32_t it = 0; it < total && ok; ++it) {
                for (int h = 0; h < 2; ++h) {                        // transform of the two x tiles of K-step `it`
                    const uint32_t xi = 2 * it + h;
                    const int xs = xi % kXStages;
                    if (!(ok = mbar_wait(&acc_empty[h], (it & 1) ^ 1, abort_flag))) break;
                    if (!(ok = mbar_wait(&x_full[xs], (xi / kXStages) & 1, abort_flag))) break;
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(smem + xs * kXTileBytes);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t adesc = rowwise ? make_smem_desc(a_addr + (ks >> 2) * kBoxBytesF + (ks & 3) * 32, 16, 1024, 2)
                                                       : make_smem_desc(a_addr + ks * 2048, kBoxBytesF, 1024, 2);
                        const uint64_t bdesc = make_smem_desc(t_addr + (ks >> 2) * kBoxBytesF + (ks & 3) * 32, 16, 1024, 2);
                        tc_mma_f16(tmem_base + kRhtCol + h * 128, adesc, bdesc, idesc_rht, ks != 0 ? 1u : 0u);
                    }
                    tc_commit(&x_empty[xs]);
                    tc_commit(&acc_full[h]);
                }
                if (ok && it >= 1) ok = main_step(it - 1);           // the product runs one K-step behind the transform
            }
            if (ok && total > 0) ok = main_step(total - 1);
            if (!ok) *abort_flag = 1;
        }
    } else if (warp >= 4 && warp < 12) {
        // ------------------------------------------------------------------ quantiser groups (h = 0: warps 4..7, h = 1: warps 8..11)
        const int h = (warp - 4) >> 2;
        const int q = warp & 3;                                  // TMEM lane quadrant
        const int row = q * 32 + lane;                           // row of the tile this thread owns
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        const float cg = p.g == 32 ? 0.17677669529663687f : p.g == 128 ? 0.08838834764831845f : 1.0f;
        bool ok = true;
        int mt = 0, nt = 0;
        for (uint32_t it = 0; it < total; ++it) {
            const int kt = (int)(it % (uint32_t)num_kt);
            if (kt == 0) tile_coords_f((int)(blockIdx.x + (it / (uint32_t)num_kt) * gridDim.x), p.m_tiles, p.n_tiles, mt, nt);
            const int s = it % kStagesF;
            ok = mbar_wait(&acc_full[h], it & 1, abort_flag) && mbar_wait(&stage_empty[s], ((it / kStagesF) & 1) ^ 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            // linear index of this thread's first element in the full K-major operand: keys the SR draws
            const uint64_t i0 = (uint64_t)((int64_t)mt * FM + row) * (uint64_t)p.K + (uint64_t)(kt * 256 + 128 * h);
            uint8_t* code_row = smem_a4 + s * kA4Bytes + row * 128;
            uint32_t sb_all = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t raw[32], rw[8] = {0u, 0u, 0u, 0u, 0u, 0u, 0u, 0u}, packed[4], sb = 0;
                float y[32];
                tmem_ld_32x32b_x32(tmem_base + lane_base + kRhtCol + h * 128 + 32 * j, raw);
                tmem_ld_wait();
                if (j == 3) {                                    // the transform accumulator is free once it has been read
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[h]);
                }
                if (ROUNDING != 1) sr_draws32(p.keys, p.stream_tag, i0 + 32 * j, rw);
#pragma unroll
                for (int i = 0; i < 32; ++i) y[i] = __uint_as_float(raw[i]) * cg;
                quantize_block32_rw<ROUNDING>(y, rw, packed, sb, p.pipe);
                // MX block j of this half = 16-byte chunk 4 h + j of the row, 128-byte swizzle
                *reinterpret_cast<uint4*>(code_row + ((((4 * h + j) ^ (row & 7))) << 4)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                sb_all |= sb << (8 * j);
            }
            // scale image of this half: 128 rows x 4 K-blocks in the tcgen05 tiling
            uint8_t* sf_stage = smem_sf + s * kSfStageF;
            *reinterpret_cast<uint32_t*>(sf_stage + h * kSfTileF + lane * 16 + q * 4) = sb_all;
            fence_proxy_async_smem();                            // the codes are read by the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(&grp_bar[h]);
            ok = mbar_wait(&grp_bar[h], it & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            // every warp copies the image into its own TMEM lane quadrant (the MMA wants it in all four)
            const uint32_t sf_t = tmem_base + lane_base + kSfColF + s * kSfSlotColsF;
            tmem_st_32x32b_x4(sf_t + 4 * h, reinterpret_cast<const uint4*>(sf_stage + h * kSfTileF)[lane]);
            if (h == 0) {                                        // the B scales of this K-step (two tiles)
                ok = mbar_wait(&b_full[s], (it / kStagesF) & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint4* sfb = reinterpret_cast<const uint4*>(sf_stage + 2 * kSfTileF);
                tmem_st_32x32b_x8(sf_t + 8, sfb[lane], sfb[32 + lane]);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&a_full[s]);
        }
        if (!ok && lane == 0) *abort_flag = 1;
    } else if (warp >= 12) {
        // ------------------------------------------------------------------ epilogue (warps 12..15)
        const int q = warp & 3;
        uint32_t tile_i = 0;
        bool ok = true;
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
                tmem_ld_32x32b_x32(tmem_base + kMainCol + ((uint32_t)(q * 32) << 16) + c * 32, r);
                tmem_ld_wait();
                const int64_t col = col0 + c * 32;
                if (row < p.M && col < p.N) {
                    const int nvalid = (int)min((int64_t)32, p.N - col);      // multiple of 8
                    if (p.out_fp32) {
                        float* dst = static_cast<float*>(p.C) + row * p.ldc + col;
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            if (4 * v < nvalid)
                                reinterpret_cast<float4*>(dst)[v] = make_float4(__uint_as_float(r[4 * v]) * p.alpha, __uint_as_float(r[4 * v + 1]) * p.alpha,
                                                                                __uint_as_float(r[4 * v + 2]) * p.alpha, __uint_as_float(r[4 * v + 3]) * p.alpha);
                    } else {
                        __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.C) + row * p.ldc + col;
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            if (8 * v < nvalid) {
                                uint32_t w[4];
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(r[8 * v + 2 * j]) * p.alpha,
                                                                                    __uint_as_float(r[8 * v + 2 * j + 1]) * p.alpha);
                                    w[j] = *reinterpret_cast<const uint32_t*>(&hh);
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
        // A wait expired somewhere: give copies still in flight time to land before the CTA's shared memory goes away.
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace

cudaError_t fetch_gemm_fused_status(unsigned int* word) { return device_status_fetch(word); }

cudaError_t gemm_fused_init() {
    const void* kernels[3] = {(const void*)gemm_fused_kernel<0>, (const void*)gemm_fused_kernel<1>, (const void*)gemm_fused_kernel<2>};
    for (const void* k : kernels) {
        const cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemF);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

bool gemm_fused_eligible(const FusedGemmArgs& a) {
    return (a.g == 32 || a.g == 64 || a.g == 128) && a.K % 256 == 0 && a.has_tmap_x;
}

cudaError_t launch_gemm_fused(const FusedGemmArgs& a, cudaStream_t stream) {
    FParams p;
    p.sfb = a.sfb; p.C = a.C;
    p.M = a.M; p.N = a.N; p.K = a.K; p.ldc = a.ldc;
    p.alpha = a.alpha; p.out_fp32 = a.out_fp32;
    p.m_tiles = (int)((a.M + FM - 1) / FM);
    p.n_tiles = (int)((a.N + FN - 1) / FN);
    p.g = a.g; p.reduce_dim = a.reduce_dim; p.stream_tag = a.stream_tag; p.seed = a.seed;
    p.pipe = make_pipe_consts();
    {
        uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);
        for (int i = 0; i < 10; ++i) {
            p.keys.k0[i] = k0; p.keys.k1[i] = k1;
            k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
        }
    }
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int tiles = p.m_tiles * p.n_tiles;
    const int grid = tiles < sms ? tiles : sms;
    if (a.rounding == 0) gemm_fused_kernel<0><<<grid, kThreadsF, kSmemF, stream>>>(a.tmap_x, a.tmap_b, p);
    else if (a.rounding == 2) gemm_fused_kernel<2><<<grid, kThreadsF, kSmemF, stream>>>(a.tmap_x, a.tmap_b, p);
    else gemm_fused_kernel<1><<<grid, kThreadsF, kSmemF, stream>>>(a.tmap_x, a.tmap_b, p);
    return cudaGetLastError();
}

}  // namespace mx
