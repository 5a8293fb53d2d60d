// Block-scaled FP4 GEMM, CTA-pair variant (tcgen05 cta_group::2): two CTAs of a 2-CTA cluster share one 256 x 256
// output tile.  Each CTA loads 128 rows of A and only HALF of the B tile (128 of its 256 rows); the pair MMA reads
// both halves, so per MMA a tensor core pulls 4 KB + 4 KB from its own shared memory instead of 4 KB + 8 KB.  The
// 1-CTA kernel (gemm.cu) is bound by exactly that operand traffic.  Each CTA keeps the accumulator of its own 128
// rows (all 256 columns) in its TMEM.
//
// The scale tiles travel in their own, deeper ring (8 slots, decoupled from the 6 operand stages), so they are in
// TMEM long before the MMAs that need them; the only tight loop left is the reuse of an operand stage.
//
// Roles per CTA (11 warps), all waits bounded as in gemm.cu:
//   warp 0      TMA producer: own A rows, own half of B (completion counted on the LEADER's barrier);
//   warp 10     scale loader: own A-row scale tiles and the scale tiles of all 256 B rows, bulk copies into the ring;
//   warp 1      MMA issuer, leader CTA only: four K = 64 pair-MMAs per stage; tcgen05.commit frees stage, scale slot
//               and accumulator in BOTH CTAs;
//   warps 2..5  epilogue of the CTA's own 128 x 256 half tile;
//   warps 6..9  scale movers: shared memory -> registers -> own TMEM (tcgen05.st), then arrive on the leader's barrier.
// A-row scales are per CTA; every CTA needs the scales of all 256 B rows.
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx.cuh"

namespace mx {
namespace {

constexpr int PM = 256, PN = 256;                           // pair tile
constexpr int kStagesP = 6;
constexpr uint32_t kAB = 128 * kGemmBKBytes;                // 16 KB: 128 rows x 128 B, for A and for the B half
constexpr uint32_t kSfTile = 512;
constexpr uint32_t kSfaB = 2 * kSfTile;                     // own 128 A rows, 2 tiles (8 K-blocks) per stage
constexpr uint32_t kSfbB = 2 * 2 * kSfTile;                 // all 256 B rows
constexpr uint32_t kStageB = 2 * kAB;                       // 32 KB: A rows + B half
constexpr int kSfSlotsP = kStagesP;                         // scale ring: shared-memory slot i feeds TMEM slot i; same ring
                                                            // index as the operand stages so ONE commit frees both
constexpr uint32_t kSfSlotB = kSfaB + kSfbB;                // 3 KB
constexpr uint32_t kSmemP = kStagesP * kStageB + kSfSlotsP * kSfSlotB + 1024 + 512;
constexpr uint32_t kAccColP = 0, kSfColP = 256, kSfSlotColsP = 24;
constexpr int kGroupMP = 8;                                 // rasterisation: 8 pair-tiles (2048 rows) share B tiles in L2
constexpr int kThreadsP = 11 * 32;

struct ParamsP {
    const uint8_t* sfa;
    const uint8_t* sfb;
    void* C;
    int64_t M, N, K, ldc;
    float alpha;
    int out_fp32;
    int m_tiles, n_tiles;                                   // in pair tiles
};

__device__ __forceinline__ void tile_coords_p(int t, int m_tiles, int n_tiles, int& mt, int& nt) {
    const int per_group = kGroupMP * n_tiles;
    const int grp = t / per_group;
    const int first_m = grp * kGroupMP;
    const int gm = min(kGroupMP, m_tiles - first_m);
    const int r = t - grp * per_group;
    mt = first_m + r % gm;
    nt = r / gm;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreadsP, 1)
gemm_mxf4_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b, const ParamsP p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sf_ring = smem + kStagesP * kStageB;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sf_ring + kSfSlotsP * kSfSlotB);
    uint64_t* full_bar = bars;                              // [kStagesP] leader: A and B halves of both CTAs landed
    uint64_t* empty_bar = full_bar + kStagesP;              // [kStagesP] per CTA: stage free (pair commit)
    uint64_t* sfl_full = empty_bar + kStagesP;              // [kSfSlotsP] per CTA: scale tiles landed in the ring slot
    uint64_t* sf_full = sfl_full + kSfSlotsP;                // [kSfSlotsP] leader: scales of both CTAs are in TMEM
    uint64_t* sf_empty = sf_full + kSfSlotsP;               // [kSfSlotsP] per CTA: scale slot free (pair commit)
    uint64_t* tmem_full = sf_empty + kSfSlotsP;             // per CTA: accumulator complete (pair commit)
    uint64_t* tmem_empty = tmem_full + 1;                   // leader: both CTAs drained their accumulators
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                // 0 = leader
    const uint32_t pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_tiles = p.m_tiles * p.n_tiles;
    const int nkc = (int)(p.K >> 7);                        // 128-element scale tiles along K
    const int num_kt = (nkc + 1) >> 1;                      // 256-element pipeline steps
    const uint32_t my_tiles = pair < (uint32_t)num_tiles ? ((uint32_t)num_tiles - pair + num_pairs - 1) / num_pairs : 0u;
    const uint32_t total = my_tiles * (uint32_t)num_kt;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStagesP; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int s = 0; s < kSfSlotsP; ++s) { mbar_init(&sfl_full[s], 1); mbar_init(&sf_full[s], 8); mbar_init(&sf_empty[s], 1); }
        mbar_init(tmem_full, 1);
        mbar_init(tmem_empty, 8);
        *abort_flag = 0;
        mbar_fence_init();
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, 512);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                     // both CTAs' barriers exist before anyone signals across
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (uint32_t tl = 0; tl < my_tiles && ok; ++tl) {
                int mt, nt;
                tile_coords_p((int)(pair + tl * num_pairs), p.m_tiles, p.n_tiles, mt, nt);
                const int a_rt = 2 * mt + (int)rank;                            // this CTA's 128-row tile of A
                for (int kt = 0; kt < num_kt; ++kt, ++it) {
                    const int s = it % kStagesP;
                    if (!(ok = mbar_wait(&empty_bar[s], ((it / kStagesP) & 1) ^ 1, abort_flag))) break;
                    uint8_t* st = smem + s * kStageB;
                    if (rank == 0) mbar_expect_tx(&full_bar[s], 4 * kAB);       // two loads from each CTA
                    tma_load_2d_pair(st, &tmap_a, &full_bar[s], kt * kGemmBKBytes, a_rt * 128);
                    tma_load_2d_pair(st + kAB, &tmap_b, &full_bar[s], kt * kGemmBKBytes, nt * PN + (int)rank * 128);
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            // instruction descriptor: A, B = E2M1 (1), scale = UE8M0 (1), K-major, N >> 3 at bit 17, M >> 4 at bit 24
            const uint32_t idesc_base = (1u << 7) | (1u << 10) | ((uint32_t)(PN >> 3) << 17) | (1u << 23) | ((uint32_t)(PM >> 4) << 24);
            uint32_t tile_i = 0;
            bool ok = true;
            for (uint32_t it = 0; it < total; ++it) {
                const int kt = (int)(it % (uint32_t)num_kt);
                const int s = it % kStagesP, slot = it % kSfSlotsP;
                if (kt == 0) {
                    if (!(ok = mbar_wait(tmem_empty, (tile_i & 1) ^ 1, abort_flag))) break;
                }
                if (!(ok = mbar_wait(&full_bar[s], (it / kStagesP) & 1, abort_flag))) break;
                if (!(ok = mbar_wait(&sf_full[slot], (it / kSfSlotsP) & 1, abort_flag))) break;
                tc_fence_after_sync();
                const uint32_t st = smem_u32(smem + s * kStageB);
                const int nch = min(2, nkc - 2 * kt);
                const uint32_t sfa_t = tmem_base + kSfColP + slot * kSfSlotColsP, sfb_t = sfa_t + 8;
                for (int kb = 0; kb < 2 * nch; ++kb) {
                    const uint64_t adesc = make_smem_desc(st + kb * 32, 16, 1024, 2);
                    const uint64_t bdesc = make_smem_desc(st + kAB + kb * 32, 16, 1024, 2);
                    const uint32_t sf_id = (uint32_t)(kb & 1) * 2u;
                    const uint32_t idesc = idesc_base | (sf_id << 29) | (sf_id << 4);
                    tc_mma_mxf4_pair(tmem_base + kAccColP, adesc, bdesc, idesc,
                                     (sfa_t + 4 * (kb >> 1)) | (sf_id << 30), (sfb_t + 8 * (kb >> 1)) | (sf_id << 30),
                                     (kt | kb) != 0 ? 1u : 0u);
                }
                tc_commit_pair(&empty_bar[s]);                                 // frees the operand stage and the scale slot
                if (kt == num_kt - 1) { tc_commit_pair(tmem_full); ++tile_i; }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp == 10) {
        // ------------------------------------------------------------------ scale loader (both CTAs)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (uint32_t tl = 0; tl < my_tiles && ok; ++tl) {
                int mt, nt;
                tile_coords_p((int)(pair + tl * num_pairs), p.m_tiles, p.n_tiles, mt, nt);
                const int a_rt = 2 * mt + (int)rank;
                const bool has_a = (int64_t)a_rt * 128 < p.M;
                const int n_row_tiles = min(2, (int)((p.N - (int64_t)nt * PN + 127) >> 7));
                for (int kt = 0; kt < num_kt; ++kt, ++it) {
                    const int slot = it % kSfSlotsP;
                    // the slot's previous scales (shared memory and TMEM) are dead once the MMAs that read them completed
                    if (!(ok = mbar_wait(&empty_bar[slot], ((it / kSfSlotsP) & 1) ^ 1, abort_flag))) break;
                    uint8_t* dst = sf_ring + slot * kSfSlotB;
                    const int nch = min(2, nkc - 2 * kt);
                    mbar_expect_tx(&sfl_full[slot], (uint32_t)nch * kSfTile * ((has_a ? 1u : 0u) + (uint32_t)n_row_tiles));
                    if (has_a) bulk_load(dst, p.sfa + ((int64_t)a_rt * nkc + 2 * kt) * kSfTile, nch * kSfTile, &sfl_full[slot]);
                    for (int j = 0; j < n_row_tiles; ++j)
                        bulk_load(dst + kSfaB + j * 2 * kSfTile, p.sfb + ((int64_t)(nt * 2 + j) * nkc + 2 * kt) * kSfTile,
                                  nch * kSfTile, &sfl_full[slot]);
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp >= 6) {
        // ------------------------------------------------------------------ scale movers (both CTAs, warps 6..9)
        const int q = warp & 3;
        const uint32_t lane_base = (uint32_t)(q * 32) << 16;
        bool ok = true;
        for (uint32_t it = 0; it < total; ++it) {
            const int slot = it % kSfSlotsP;
            if (lane == 0) ok = mbar_wait(&sfl_full[slot], (it / kSfSlotsP) & 1, abort_flag);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            tc_fence_after_sync();
            const uint4* sf = reinterpret_cast<const uint4*>(sf_ring + slot * kSfSlotB) + lane;          // 32 uint4 per tile
            const uint32_t sfa_t = tmem_base + lane_base + kSfColP + slot * kSfSlotColsP, sfb_t = sfa_t + 8;
            tmem_st_32x32b_x8(sfa_t, sf[0], sf[32]);
            tmem_st_32x32b_x16(sfb_t, sf[64], sf[128], sf[96], sf[160]);
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(&sf_full[slot], 0);
        }
        if (!ok && lane == 0) *abort_flag = 1;
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
        const int q = warp & 3;
        bool ok = true;
        for (uint32_t tl = 0; tl < my_tiles; ++tl) {
            int mt, nt;
            tile_coords_p((int)(pair + tl * num_pairs), p.m_tiles, p.n_tiles, mt, nt);
            if (lane == 0) ok = mbar_wait(tmem_full, tl & 1, abort_flag);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            tc_fence_after_sync();
            const int64_t row = (int64_t)mt * PM + (int64_t)rank * 128 + q * 32 + lane;
            const int64_t col0 = (int64_t)nt * PN;
#pragma unroll 1
            for (int c = 0; c < PN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(tmem_base + kAccColP + ((uint32_t)(q * 32) << 16) + c * 32, r);
                tmem_ld_wait();
                const int64_t col = col0 + c * 32;
                if (row < p.M && col < p.N) {
                    const int nvalid = (int)min((int64_t)32, p.N - col);      // multiple of 8
                    if (p.out_fp32) {
                        float* dst = static_cast<float*>(p.C) + row * p.ldc + col;
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            if (4 * v < nvalid)
                                reinterpret_cast<float4*>(dst)[v] =
                                    make_float4(__uint_as_float(r[4 * v]) * p.alpha, __uint_as_float(r[4 * v + 1]) * p.alpha,
                                                __uint_as_float(r[4 * v + 2]) * p.alpha, __uint_as_float(r[4 * v + 3]) * p.alpha);
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
            if (lane == 0) mbar_arrive_cluster(tmem_empty, 0);
        }
        if (!ok && lane == 0) *abort_flag = 1;
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);      // let copies in flight land
        __syncthreads();
    }
    cluster_sync_all();                                     // neither CTA leaves while the other may still signal it
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

}  // namespace

cudaError_t gemm_pair_init() {
    return cudaFuncSetAttribute(gemm_mxf4_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemP);
}

cudaError_t launch_gemm_pair(const GemmArgs& a, cudaStream_t stream) {
    ParamsP p;
    p.sfa = a.sfa; p.sfb = a.sfb; p.C = a.C;
    p.M = a.M; p.N = a.N; p.K = a.K; p.ldc = a.ldc;
    p.alpha = a.alpha; p.out_fp32 = a.out_fp32;
    p.m_tiles = (int)((a.M + PM - 1) / PM);
    p.n_tiles = (int)((a.N + PN - 1) / PN);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int tiles = p.m_tiles * p.n_tiles;
    const int pairs = tiles < sms / 2 ? tiles : sms / 2;
    gemm_mxf4_pair_kernel<<<2 * pairs, kThreadsP, kSmemP, stream>>>(a.tmap_a, a.tmap_b_half, p);
    return cudaGetLastError();
}

}  // namespace mx
