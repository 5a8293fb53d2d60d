// Block-scaled FP4 GEMM on the 5th-generation tensor cores (MXFP4_GEMM of Algorithm 3):
//     C[M, N] = alpha * sum_k deq(A)[i, k] deq(B)[j, k]
// tcgen05.mma kind::mxf4 (E2M1 x E2M1, one UE8M0 scale per 32 elements along K, fp32 accumulation in TMEM).
//
// Persistent, warp-specialised kernel, one CTA per SM, 128 x 256 output tile:
//   warp 0      TMA producer: per stage 128 B (256 elements) of K for 128 rows of A and 256 rows of B through
//               128-byte-swizzled tensor maps, plus the scale tiles (already in the tcgen05 tiling in global
//               memory) as plain bulk copies;
//   warp 1      MMA issuer: four K = 64 MMAs per stage;
//   warps 2..5  epilogue: TMEM -> registers (tcgen05.ld) -> alpha -> bf16/fp32 -> global;
//   warps 6..9  scale-factor movers: per stage, shared memory -> registers -> TMEM (tcgen05.st), one warp per
//               TMEM lane quadrant (the MMA wants the scales replicated in all four).  Doing this with
//               tcgen05.cp from the MMA thread put ~64 cycles per copy in series with the MMAs (six per step:
//               measured 3.6 vs 5.25 PFLOP/s without them); tcgen05.st runs beside the MMA pipe.
// Every mbarrier wait is bounded; on expiry the CTA records a status word and unwinds.
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx.cuh"

namespace mx {

namespace {

constexpr int BM = kGemmBM, BN = kGemmBN;
constexpr int kStages = 4;
constexpr uint32_t kABytes = BM * kGemmBKBytes;             // 16 KB
constexpr uint32_t kBBytes = BN * kGemmBKBytes;             // 32 KB
constexpr uint32_t kSfChunk = 512;                          // scale tile: 128 rows x 4 K-blocks
constexpr uint32_t kSfaBytes = 2 * kSfChunk;                // 2 tiles per stage (8 K-blocks)
constexpr uint32_t kSfbBytes = (BN / 128) * 2 * kSfChunk;
constexpr uint32_t kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;   // 51 KB, multiple of 1024
constexpr uint32_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kAccCol = 0;                             // 256 fp32 accumulator columns
constexpr uint32_t kSfCol = 256;                            // kSfSlots slots of (8 SFA + 16 SFB) columns
constexpr uint32_t kSfSlotCols = 24;
constexpr int kSfSlots = kStages;                           // scale slot i belongs to stage i: one commit frees both
constexpr int kGroupM = 16;                                 // tile rasterisation: 16 m-tiles share B tiles in L2
constexpr int kThreads = 10 * 32;

struct Params {
    const uint8_t* sfa;
    const uint8_t* sfb;
    void* C;
    int64_t M, N, K, ldc;
    float alpha;
    int out_fp32;
    int accumulate;                                         // fp32 output only: C += instead of C =
    int m_tiles, n_tiles;
};

__device__ __forceinline__ void tile_coords(int t, int m_tiles, int n_tiles, int& mt, int& nt) {
    const int per_group = kGroupM * n_tiles;
    const int grp = t / per_group;
    const int first_m = grp * kGroupM;
    const int gm = min(kGroupM, m_tiles - first_m);
    const int r = t - grp * per_group;
    mt = first_m + r % gm;
    nt = r / gm;
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_mxf4_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
    uint64_t* full_bar = bars;                              // [kStages]  TMA -> MMA, scale movers
    uint64_t* empty_bar = full_bar + kStages;               // [kStages]  MMA -> TMA
    uint64_t* sf_full = empty_bar + kStages;                // [kSfSlots] scale movers -> MMA
    uint64_t* tmem_full = sf_full + kSfSlots;               // MMA -> epilogue
    uint64_t* tmem_empty = tmem_full + 1;                   // epilogue -> MMA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_tiles = p.m_tiles * p.n_tiles;
    const int nkc = (int)(p.K >> 7);                          // 128-element scale chunks along K
    const int num_kt = (nkc + 1) >> 1;                        // 256-element pipeline steps
    const uint32_t my_tiles = blockIdx.x < (uint32_t)num_tiles ? ((uint32_t)num_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0u;
    const uint32_t total = my_tiles * (uint32_t)num_kt;       // K-steps this CTA runs, over all its tiles

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int s = 0; s < kSfSlots; ++s) mbar_init(&sf_full[s], 4);
        mbar_init(tmem_full, 1);
        mbar_init(tmem_empty, 4);
        *abort_flag = 0;
        mbar_fence_init();
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
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
                tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
                const int n_row_tiles = min(BN / 128, (int)((p.N - (int64_t)nt * BN + 127) >> 7));
                for (int kt = 0; kt < num_kt; ++kt, ++it) {
                    const int s = it % kStages;
                    const uint32_t ph = (it / kStages) & 1;
                    if (!(ok = mbar_wait(&empty_bar[s], ph ^ 1, abort_flag))) break;
                    uint8_t* st = smem + s * kStageBytes;
                    const int nch = min(2, nkc - 2 * kt);
                    mbar_expect_tx(&full_bar[s], kABytes + kBBytes + nch * kSfChunk * (1 + n_row_tiles));
                    tma_load_2d(st, &tmap_a, &full_bar[s], kt * kGemmBKBytes, mt * BM);
                    tma_load_2d(st + kABytes, &tmap_b, &full_bar[s], kt * kGemmBKBytes, nt * BN);
                    bulk_load(st + kABytes + kBBytes, p.sfa + ((int64_t)mt * nkc + 2 * kt) * kSfChunk, nch * kSfChunk, &full_bar[s]);
                    for (int j = 0; j < n_row_tiles; ++j)
                        bulk_load(st + kABytes + kBBytes + kSfaBytes + j * 2 * kSfChunk,
                                  p.sfb + ((int64_t)(nt * (BN / 128) + j) * nkc + 2 * kt) * kSfChunk, nch * kSfChunk, &full_bar[s]);
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // instruction descriptor: A, B = E2M1 (1), scale = UE8M0 (1), K-major, N >> 3 at bit 17, M >> 4 at bit 24
            const uint32_t idesc_base = (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | (1u << 23) | ((uint32_t)(BM >> 4) << 24);
            uint32_t tile_i = 0;
            bool ok = true;
            for (uint32_t it = 0; it < total; ++it) {
                const int kt = (int)(it % (uint32_t)num_kt);
                const int s = it % kStages, slot = it % kSfSlots;
                if (kt == 0) {
                    if (!(ok = mbar_wait(tmem_empty, (tile_i & 1) ^ 1, abort_flag))) break;
                }
                if (!(ok = mbar_wait(&full_bar[s], (it / kStages) & 1, abort_flag))) break;
                if (!(ok = mbar_wait(&sf_full[slot], (it / kSfSlots) & 1, abort_flag))) break;
                tc_fence_after_sync();
                const uint32_t st = smem_u32(smem + s * kStageBytes);
                const int nch = min(2, nkc - 2 * kt);
                const uint32_t sfa_t = tmem_base + kSfCol + slot * kSfSlotCols, sfb_t = sfa_t + 8;
                for (int kb = 0; kb < 2 * nch; ++kb) {
                    const uint64_t adesc = make_smem_desc(st + kb * 32, 16, 1024, 2);
                    const uint64_t bdesc = make_smem_desc(st + kABytes + kb * 32, 16, 1024, 2);
                    const uint32_t sf_id = (uint32_t)(kb & 1) * 2u;           // byte pair inside the 32-bit scale column
                    const uint32_t idesc = idesc_base | (sf_id << 29) | (sf_id << 4);
                    tc_mma_mxf4(tmem_base + kAccCol, adesc, bdesc, idesc,
                                (sfa_t + 4 * (kb >> 1)) | (sf_id << 30), (sfb_t + 8 * (kb >> 1)) | (sf_id << 30),
                                (kt | kb) != 0 ? 1u : 0u);
                }
                tc_commit(&empty_bar[s]);                // one commit frees the stage and its scale slot (same ring index)
                if (kt == num_kt - 1) { tc_commit(tmem_full); ++tile_i; }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp >= 6) {
        // ------------------------------------------------------------------ scale-factor movers (warps 6..9)
        // A 512-byte scale tile is the image of 32 TMEM lanes x 4 columns: lane l holds the 16 bytes at l * 16
        // (rows l, l+32, l+64, l+96 of the 128-row tile, four K-blocks each).  Each warp writes that image into
        // its own lane quadrant, which gives the four-fold replication the MMA expects.  Tiles the stage does
        // not hold (K tail, N tail) leave stale bytes in columns whose products are never stored.
        const int q = warp & 3;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        bool ok = true;
        for (uint32_t it = 0; it < total; ++it) {
            const int s = it % kStages, slot = it % kSfSlots;
            ok = mbar_wait(&full_bar[s], (it / kStages) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const uint4* sf = reinterpret_cast<const uint4*>(smem + s * kStageBytes + kABytes + kBBytes) + lane;   // 32 uint4 per tile
            const uint32_t sfa_t = tmem_base + lane_base + kSfCol + slot * kSfSlotCols, sfb_t = sfa_t + 8;
            // stage layout: SFA tile 0, 1 | SFB (rows 0-127) tile 0, 1 | SFB (rows 128-255) tile 0, 1
            tmem_st_32x32b_x8(sfa_t, sf[0], sf[32]);
            tmem_st_32x32b_x16(sfb_t, sf[64], sf[128], sf[96], sf[160]);      // columns: (tile 0: rows 0-127 | 128-255) | (tile 1: ...)
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sf_full[slot]);
        }
        if (!ok && lane == 0) *abort_flag = 1;
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;                                   // TMEM lane quadrant this warp may read
        uint32_t tile_i = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++tile_i) {
            int mt, nt;
            tile_coords(t, p.m_tiles, p.n_tiles, mt, nt);
            ok = mbar_wait(tmem_full, tile_i & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const int64_t row = (int64_t)mt * BM + q * 32 + lane;
            const int64_t col0 = (int64_t)nt * BN;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(tmem_base + kAccCol + ((uint32_t)(q * 32) << 16) + c * 32, r);
                tmem_ld_wait();
                const int64_t col = col0 + c * 32;
                if (row < p.M && col < p.N) {
                    const int nvalid = (int)min((int64_t)32, p.N - col);      // multiple of 8
                    if (p.out_fp32) {
                        float* dst = static_cast<float*>(p.C) + row * p.ldc + col;
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            if (4 * v < nvalid) {
                                float4 o = p.accumulate ? reinterpret_cast<const float4*>(dst)[v] : make_float4(0.f, 0.f, 0.f, 0.f);
                                // product rounded first, then one add: the same two roundings as the TMA-reduce path (no fused multiply-add)
                                o.x = __fadd_rn(o.x, __fmul_rn(__uint_as_float(r[4 * v]), p.alpha));
                                o.y = __fadd_rn(o.y, __fmul_rn(__uint_as_float(r[4 * v + 1]), p.alpha));
                                o.z = __fadd_rn(o.z, __fmul_rn(__uint_as_float(r[4 * v + 2]), p.alpha));
                                o.w = __fadd_rn(o.w, __fmul_rn(__uint_as_float(r[4 * v + 3]), p.alpha));
                                reinterpret_cast<float4*>(dst)[v] = o;
                            }
                    } else {
                        __nv_bfloat16* dst = static_cast<__nv_bfloat16*>(p.C) + row * p.ldc + col;
#pragma unroll
                        for (int v = 0; v < 4; ++v)
                            if (8 * v < nvalid) {
                                uint32_t w[4];
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * v + 2 * j]) * p.alpha,
                                                                                   __uint_as_float(r[8 * v + 2 * j + 1]) * p.alpha);
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
        // A wait expired somewhere: give copies still in flight time to land before the CTA's shared memory goes away.
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

cudaError_t fetch_gemm_status(unsigned int* word) { return device_status_fetch(word); }

cudaError_t gemm_init() {
    return cudaFuncSetAttribute(gemm_mxf4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
}

cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t stream) {
    Params p;
    p.sfa = a.sfa; p.sfb = a.sfb; p.C = a.C;
    p.M = a.M; p.N = a.N; p.K = a.K; p.ldc = a.ldc;
    p.alpha = a.alpha; p.out_fp32 = a.out_fp32; p.accumulate = a.accumulate;
    p.m_tiles = (int)((a.M + BM - 1) / BM);
    p.n_tiles = (int)((a.N + BN - 1) / BN);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int tiles = p.m_tiles * p.n_tiles;
    const int grid = tiles < sms ? tiles : sms;
    gemm_mxf4_kernel<<<grid, kThreads, kSmemBytes, stream>>>(a.tmap_a, a.tmap_b, p);
    return cudaGetLastError();
}

}  // namespace mx
