// Block-scaled FP4 GEMM, CTA-pair variant (tcgen05 cta_group::2): two CTAs of a 2-CTA cluster share one 256 x 256
// output tile.  Each CTA loads 128 rows of A and only HALF of the B tile (128 of its 256 rows); the pair MMA reads
// both halves, so per MMA a tensor core pulls 4 KB + 4 KB from its own shared memory instead of 4 KB + 8 KB.  The
// 1-CTA kernel (gemm.cu) is bound by exactly that operand traffic.  Each CTA keeps the accumulator of its own 128
// rows (all 256 columns) in its TMEM.
//
// Shared memory (all 227 KB): six operand stages of 32 KB, a six-slot scale ring of 3 KB, 16 KB of epilogue staging.
// TMEM: 256 accumulator columns + six scale slots of 24 columns.
//
// Roles per CTA (12 warps in three warp groups), all waits bounded as in gemm.cu:
//   warp 0       TMA producer: own A rows, own half of B (completion counted on the LEADER's barrier);
//   warp 3       scale loader: own A-row scale tiles and the scale tiles of all 256 B rows, bulk copies into ring slot
//                s of stage s (free again when the step's MMAs, and with them its scale copies, have completed);
//   warps 1, 2   MMA issuers, leader CTA only, taking the K-steps in turn under a baton.  Per step: six tcgen05.cp
//                carry the step's scale tiles from the ring into TMEM slot s of BOTH CTAs (the copy itself replicates
//                them to the four lane quadrants and reads shared memory once; they are issued while the other
//                thread still issues its MMAs), then four K = 64 pair-MMAs; ONE multicast tcgen05.commit per step
//                frees operand stage, ring slot and TMEM scale slot in both CTAs;
//   warp 8       forwards "this CTA's scale tiles of step i have landed" to the leader's full barrier of the stage,
//                the same one the operand bytes complete, so the issuer waits once (warps 9..11 only fill the group);
//   warps 4..7   epilogue of the CTA's own 128 x 256 half tile: accumulator -> registers (packed bf16) -> hand the
//                accumulator back -> swizzled staging -> TMA stores (or reduce-adds when accumulating).
// A-row scales are per CTA; every CTA needs the scales of all 256 B rows.
#include <cuda_bf16.h>

#include <cstdlib>

#include "kernels.h"
#include "ptx.cuh"

namespace mx {
namespace {

constexpr int PM = 256, PN = 256;                           // pair tile
constexpr uint32_t kAB = 128 * kGemmBKBytes;                // 16 KB: 128 rows x 128 B, for A and for the B half
constexpr uint32_t kSfTile = 512;
constexpr uint32_t kSfaB = 2 * kSfTile;                     // own 128 A rows, 2 tiles (8 K-blocks) per stage
constexpr uint32_t kSfbB = 2 * 2 * kSfTile;                 // all 256 B rows
constexpr uint32_t kStageB = 2 * kAB;                       // 32 KB: A rows + B half
constexpr uint32_t kSfSlotB = kSfaB + kSfbB;                // 3 KB
constexpr uint32_t kEpiBuf = 2048;                          // epilogue staging: 32 rows x 64 B, two buffers per epilogue warp (4 warps)
constexpr uint32_t kEpiB = 4 * 2 * kEpiBuf;
constexpr uint32_t kBarB = 256;
constexpr uint32_t kSfSlotColsP = 24;
constexpr int kThreadsP = 12 * 32;

// Two builds of the kernel.  FULL owns its SMs: six operand stages (all 227 KB of shared memory), one 512-column TMEM
// allocation, every register of the SM.  LITE leaves room for a second, independent kernel on the same SM (the
// tensor-core quantiser's small build, quantize_tc.cu, which quantises the OTHER product's operands meanwhile): four
// stages, TMEM taken as 256 + 128 columns, 112 registers per thread at launch.
template <bool LITE>
struct PairCfg {
    static constexpr int kStages = LITE ? 4 : 6;
    static constexpr int kSfSlots = kStages;                // scale ring: shared-memory slot i feeds TMEM slot i; same ring
                                                            // index as the operand stages so ONE commit frees both
    // The dynamic shared-memory window is at least 256-byte aligned, so rounding its base up to 1024 costs at most 768 bytes.
    static constexpr uint32_t kSmem = kStages * kStageB + kSfSlots * kSfSlotB + kEpiB + kBarB + 768;
    // Register hand-over (setmaxnreg) between the three warp groups (kRegsFwd: the forwarder's group); an increase can only
    // draw on what the CTA holds at launch (threads x registers per thread), which gemm_pair_init checks: an increase
    // that cannot be met waits forever.
    static constexpr int kRegsLight = 56, kRegsFwd = LITE ? 24 : 64, kRegsEpi = 232;
    static constexpr int kLaunchRegs = LITE ? 104 : 168;    // registers per thread the CTA is given at launch
    static_assert(kSmem <= 232448, "over the 227 KB shared-memory limit");
    static_assert(kSfSlots * kSfSlotColsP <= (LITE ? 128 : 256), "scale slots do not fit their TMEM allocation");
    static_assert(kThreadsP * kLaunchRegs >= 128 * (kRegsLight + kRegsFwd + kRegsEpi), "warp groups ask for more registers than the CTA holds");
};

struct ParamsP {
    const uint8_t* sfa;
    const uint8_t* sfb;
    void* C;
    int64_t M, N, K, ldc;
    float alpha;
    int out_fp32;
    int m_tiles, n_tiles;                                   // in pair tiles
    int c_tma;                                              // C goes out through tmap_c (else plain stores)
    int accumulate;                                         // fp32 output only: C += instead of C =
    int group_m;                                            // rasterisation: this many pair-tile rows share the B tiles in L2 (launch_gemm_pair)
};

__device__ __forceinline__ void tile_coords_p(int t, int m_tiles, int n_tiles, int kGroupMP, int& mt, int& nt) {
    const int per_group = kGroupMP * n_tiles;
    const int grp = t / per_group;
    const int first_m = grp * kGroupMP;
    const int gm = min(kGroupMP, m_tiles - first_m);
    const int r = t - grp * per_group;
    mt = first_m + r % gm;
    nt = r / gm;
}

template <bool LITE>
__device__ __forceinline__ void gemm_pair_body(const CUtensorMap& tmap_a, const CUtensorMap& tmap_b, const CUtensorMap& tmap_c, const ParamsP& p) {
    using Cfg = PairCfg<LITE>;
    constexpr int kStagesP = Cfg::kStages, kSfSlotsP = Cfg::kSfSlots;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sf_ring = smem + kStagesP * kStageB;
    uint8_t* epi_ring = sf_ring + kSfSlotsP * kSfSlotB;
    uint64_t* bars = reinterpret_cast<uint64_t*>(epi_ring + kEpiB);
    uint64_t* full_bar = bars;                              // [kStagesP] leader: operands and scale tiles of both CTAs landed
                                                            //            (1 expect_tx arrival + 1 forwarder per CTA)
    uint64_t* empty_bar = full_bar + kStagesP;              // [kStagesP] per CTA: stage and scale slot free (pair commit)
    uint64_t* sfl_full = empty_bar + kStagesP;              // [kSfSlotsP] per CTA: scale tiles landed in the ring slot
    uint64_t* turn = sfl_full + kSfSlotsP;                 // [2] leader: baton between the two MMA issuers
    uint64_t* tmem_full = turn + 2;                         // per CTA: accumulator complete (pair commit)
    uint64_t* tmem_empty = tmem_full + 1;                   // leader: both CTAs drained their accumulators
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty + 1);   // [2] base columns of the TMEM allocation(s)
    volatile uint32_t* abort_flag = tmem_slot + 2;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();                // 0 = leader
    const uint32_t pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_tiles = p.m_tiles * p.n_tiles;
    const int nkc = (int)(p.K >> 7);                        // 128-element scale tiles along K
    const int num_kt = (nkc + 1) >> 1;                      // 256-element pipeline steps
    const uint32_t my_tiles = pair < (uint32_t)num_tiles ? ((uint32_t)num_tiles - pair + num_pairs - 1) / num_pairs : 0u;
    const uint32_t total = my_tiles * (uint32_t)num_kt;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStagesP; ++s) { mbar_init(&full_bar[s], 1 + 2); mbar_init(&empty_bar[s], 1); }
        for (int s = 0; s < kSfSlotsP; ++s) mbar_init(&sfl_full[s], 1);
        mbar_init(&turn[0], 1); mbar_init(&turn[1], 1);
        mbar_init(tmem_full, 1);
        mbar_init(tmem_empty, 8);
        *abort_flag = 0;
        mbar_fence_init();
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
        if (p.c_tma) prefetch_tensormap(&tmap_c);
    }
    if (warp == 1) {
        if (LITE) {                                         // accumulator and scale slots as two allocations: 128 columns stay free
            tmem_alloc_pair(&tmem_slot[0], 256);
            tmem_alloc_pair(&tmem_slot[1], 128);
        } else {
            tmem_alloc_pair(&tmem_slot[0], 512);
        }
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();                                     // both CTAs' barriers exist before anyone signals across
    tc_fence_after_sync();
    const uint32_t tmem_acc = tmem_slot[0];                 // 256 accumulator columns
    const uint32_t tmem_sf = LITE ? tmem_slot[1] : tmem_slot[0] + 256;   // scale slots of 24 columns
    // Warp group 0 (producer, issuers, scale loader) and warp group 2 (forwarder) need few registers; the epilogue
    // group takes them to hold half an accumulator row and four TMEM loads in flight.
    // Each warp group (four warps) sets its register limit once, at the head of its own branch: all four warps must
    // execute the same setmaxnreg, and the limit must dominate the code that relies on it.
    pdl_launch_dependents();                                // the next kernel of the stream may set itself up behind this one
    pdl_wait();                                             // everything above overlapped the previous kernel's tail; its data is needed now

    if (warp < 4) {
    // ============================ warp group 0: producer, two MMA issuers, scale loader (few registers each)
    reg_dealloc<Cfg::kRegsLight>();
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (uint32_t tl = 0; tl < my_tiles && ok; ++tl) {
                int mt, nt;
                tile_coords_p((int)(pair + tl * num_pairs), p.m_tiles, p.n_tiles, p.group_m, mt, nt);
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
    } else if (warp == 1 || warp == 2) {
        // ------------------------------------------------------------------ MMA issuers (leader CTA only)
        // Issuing one pair MMA occupies its thread for ~90 cycles and a commit for ~100, which is more than the
        // tensor pipe needs for the four MMAs of a step.  Two threads therefore take the steps in turn (even steps
        // warp 1, odd steps warp 2): while one issues, the other has already waited for its operands and then
        // commits.  A baton (mbarrier turn[]) keeps the MMAs in step order, so accumulation order is fixed.
        if (rank == 0 && lane == 0) {
            // instruction descriptor: A, B = E2M1 (1), scale = UE8M0 (1), K-major, N >> 3 at bit 17, M >> 4 at bit 24
            const uint32_t idesc0 = (1u << 7) | (1u << 10) | ((uint32_t)(PN >> 3) << 17) | (1u << 23) | ((uint32_t)(PM >> 4) << 24);
            const uint32_t idesc1 = idesc0 | (2u << 29) | (2u << 4);          // scale bytes 2, 3 of the 32-bit column
            const uint64_t desc0 = make_smem_desc(smem_u32(smem), 16, 1024, 2);
            const uint32_t desc_hi = (uint32_t)(desc0 >> 32);
            const uint32_t a_lo0 = (uint32_t)desc0;
            const bool k_tail = (nkc & 1) != 0;                               // last step holds 128 elements only
            const uint32_t acc = tmem_acc;
            const uint32_t me = warp == 1 ? 0u : 1u;
            uint32_t s = me % kStagesP, ph = 0, tile_i = 0, n = 0;
            int kt = (int)me;
            while (kt >= num_kt) { kt -= num_kt; ++tile_i; }
            bool ok = true;
            for (uint32_t it = me; it < total; it += 2, ++n) {
                if (!(ok = mbar_wait(&full_bar[s], ph, abort_flag))) break;
                tc_fence_after_sync();
                const uint32_t a_lo = a_lo0 + s * (kStageB >> 4), b_lo = a_lo + (kAB >> 4);
                const uint32_t sfa_t = tmem_sf + s * kSfSlotColsP, sfb_t = sfa_t + 8;
                {   // the step's scales: shared memory -> TMEM of both CTAs, replicated to the four lane quadrants by the copy;
                    // issued while the other thread still issues its MMAs (a different TMEM slot), ordered before this
                    // thread's MMAs by program order
                    const uint32_t sf_s = smem_u32(sf_ring + s * kSfSlotB);
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        tc_cp_32x128b_warpx4_pair(sfa_t + 4 * c, make_smem_desc(sf_s + c * kSfTile, 0, 128, 0));
#pragma unroll
                        for (int j = 0; j < 2; ++j)
                            tc_cp_32x128b_warpx4_pair(sfb_t + 8 * c + 4 * j, make_smem_desc(sf_s + kSfaB + (2 * j + c) * kSfTile, 0, 128, 0));
                    }
                }
                if (kt == 0) {                                                   // the copies above did not need the accumulator
                    if (!(ok = mbar_wait(tmem_empty, (tile_i & 1) ^ 1, abort_flag))) break;
                    tc_fence_after_sync();
                }
                if (!(ok = mbar_wait_spin(&turn[me], (n & 1) ^ me ^ 1, abort_flag))) break;   // the step before mine is issued
                const uint32_t hi2 = 2u << 30;
                const bool last = kt == num_kt - 1;
                auto D = [&](uint32_t lo) { return ((uint64_t)desc_hi << 32) | lo; };
                tc_mma_mxf4_pair(acc, D(a_lo), D(b_lo), idesc0, sfa_t, sfb_t, kt != 0 ? 1u : 0u);
                tc_mma_mxf4_pair(acc, D(a_lo + 2), D(b_lo + 2), idesc1, sfa_t | hi2, sfb_t | hi2, 1u);
                if (!(last && k_tail)) {
                    tc_mma_mxf4_pair(acc, D(a_lo + 4), D(b_lo + 4), idesc0, sfa_t + 4, sfb_t + 8, 1u);
                    tc_mma_mxf4_pair(acc, D(a_lo + 6), D(b_lo + 6), idesc1, (sfa_t + 4) | hi2, (sfb_t + 8) | hi2, 1u);
                }
                tc_fence_before_sync();
                mbar_arrive(&turn[me ^ 1]);                                    // pass the baton
                tc_commit_pair(&empty_bar[s]);                                 // frees the operand stage and the scale slot
                if (last) tc_commit_pair(tmem_full);
                s += 2;
                if (s >= (uint32_t)kStagesP) { s -= kStagesP; ph ^= 1; }
                kt += 2;
                while (kt >= num_kt) { kt -= num_kt; ++tile_i; }
            }
            if (!ok) *abort_flag = 1;
        }
    } else {
        // ------------------------------------------------------------------ scale loader (both CTAs)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (uint32_t tl = 0; tl < my_tiles && ok; ++tl) {
                int mt, nt;
                tile_coords_p((int)(pair + tl * num_pairs), p.m_tiles, p.n_tiles, p.group_m, mt, nt);
                const int a_rt = 2 * mt + (int)rank;
                const bool has_a = (int64_t)a_rt * 128 < p.M;
                const int n_row_tiles = min(2, (int)((p.N - (int64_t)nt * PN + 127) >> 7));
                for (int kt = 0; kt < num_kt; ++kt, ++it) {
                    const int slot = it % kSfSlotsP;
                    // the ring slot is free once the MMAs of the step that used it (and their scale copies) have completed
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
    }
    } else if (warp >= 8) {
        // ============================ warp group 2: scale forwarder (warp 8)
        reg_dealloc<Cfg::kRegsFwd>();
        // The scale copies run in both CTAs on the leader's instruction, so the leader has to know that the peer's tiles
        // have landed too: one thread per CTA passes its ring's completions on to the leader's full barrier.
        bool ok = true;
        if (warp == 8 && lane == 0) {
            for (uint32_t it = 0; it < total; ++it) {
                const int slot = it % kSfSlotsP;
                if (!(ok = mbar_wait(&sfl_full[slot], (it / kSfSlotsP) & 1, abort_flag))) break;
                mbar_arrive_cluster(&full_bar[slot], 0);
            }
        }
        if (!ok && lane == 0) *abort_flag = 1;
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
        reg_alloc<Cfg::kRegsEpi>();                                  // warp group 1 takes the registers the others gave up
        // TMEM -> registers -> (alpha, convert) -> shared memory -> TMA store.  Each warp owns the 32 accumulator
        // lanes of its quadrant and two 2 KB staging buffers (32 rows x 64 bytes, 64-byte swizzle, so the row-per-lane
        // writes are conflict-free); the accumulator is handed back as soon as its last column is in registers.
        const int q = warp & 3;
        uint8_t* stage0 = epi_ring + q * 2 * kEpiBuf;
        uint32_t n_stores = 0;                                  // bulk groups this warp committed so far
        const uint64_t pol_c = l2_policy_evict_first();         // the output is not read again here: let the operands keep L2
        bool ok = true;
        // One staged block: 16 registers = 64 bytes of this lane's row, columns [col, col + 64 B).
        auto put = [&](const uint32_t (&w)[16], int32_t col, int32_t row0, bool in_range) {
            uint8_t* buf = stage0 + (n_stores & 1) * kEpiBuf;
            if (n_stores >= 2) {                                // the store that last read this buffer must be done with it
                if (lane == 0) bulk_wait_group_read<1>();
                __syncwarp();
            }
            uint4* dst = reinterpret_cast<uint4*>(buf + lane * 64);
            const int sw = (lane >> 1) & 3;
#pragma unroll
            for (int j = 0; j < 4; ++j) dst[j ^ sw] = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                if (in_range) {
                    if (p.accumulate) tma_reduce_add_2d(&tmap_c, buf, col, row0);
                    else tma_store_2d_hint(&tmap_c, buf, col, row0, pol_c);
                }
                bulk_commit_group();
            }
            ++n_stores;
        };
        for (uint32_t tl = 0; tl < my_tiles; ++tl) {
            int mt, nt;
            tile_coords_p((int)(pair + tl * num_pairs), p.m_tiles, p.n_tiles, p.group_m, mt, nt);
            if (lane == 0) ok = mbar_wait(tmem_full, tl & 1, abort_flag);
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) break;
            tc_fence_after_sync();
            const int64_t row0 = (int64_t)mt * PM + (int64_t)rank * 128 + q * 32;
            const int64_t row = row0 + lane;
            const int64_t col0 = (int64_t)nt * PN;
            int n_chunks = PN / 32;
            if (p.c_tma && !p.out_fp32) {
                // bf16: drain the whole accumulator into registers first (packed pairs), hand it back, then store.
                uint32_t out[PN / 2];
#pragma unroll
                for (int hb = 0; hb < 2; ++hb) {                // two batches of four 32-column loads in flight together
                    uint32_t r[4][32];
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        tmem_ld_32x32b_x32(tmem_acc + ((uint32_t)(q * 32) << 16) + (4 * hb + c) * 32, r[c]);
                    tmem_ld_wait();
                    if (hb == 1) {                              // the accumulator is in registers: hand it back before converting
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(tmem_empty, 0);
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[c][2 * j]) * p.alpha,
                                                                           __uint_as_float(r[c][2 * j + 1]) * p.alpha);
                            out[16 * (4 * hb + c) + j] = *reinterpret_cast<const uint32_t*>(&h);
                        }
                }
#pragma unroll
                for (int c = 0; c < PN / 32; ++c) {
                    uint32_t w[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) w[j] = out[16 * c + j];
                    const int64_t col = col0 + c * 32;
                    put(w, (int32_t)col, (int32_t)row0, row0 < p.M && col < p.N);
                }
                n_chunks = 0;
            }
#pragma unroll 1
            for (int c = 0; c < n_chunks; ++c) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(tmem_acc + ((uint32_t)(q * 32) << 16) + c * 32, r);
                tmem_ld_wait();
                if (c == n_chunks - 1) {                        // accumulator drained: the next tile's MMAs may start
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(tmem_empty, 0);
                }
                const int64_t col = col0 + c * 32;
                if (p.c_tma) {
                    const bool in_range = row0 < p.M && col < p.N;
                    if (p.out_fp32) {
                        uint32_t w[16];
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) w[j] = __float_as_uint(__uint_as_float(r[16 * h + j]) * p.alpha);
                            put(w, (int32_t)col + 16 * h, (int32_t)row0, in_range && col + 16 * h < p.N);
                        }
                    } else {
                        uint32_t w[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[2 * j]) * p.alpha,
                                                                           __uint_as_float(r[2 * j + 1]) * p.alpha);
                            w[j] = *reinterpret_cast<const uint32_t*>(&h);
                        }
                        put(w, (int32_t)col, (int32_t)row0, in_range);
                    }
                    } else if (row < p.M && col < p.N) {
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
        }
        if (lane == 0) bulk_wait_group<0>();                         // every store has left shared memory and is visible
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
        if (LITE) {
            tmem_dealloc_pair(tmem_slot[1], 128);
            tmem_dealloc_pair(tmem_slot[0], 256);
        } else {
            tmem_dealloc_pair(tmem_slot[0], 512);
        }
    }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreadsP, 1)
gemm_mxf4_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                      const __grid_constant__ CUtensorMap tmap_c, const ParamsP p) {
    gemm_pair_body<false>(tmap_a, tmap_b, tmap_c, p);
}

// The small-footprint build (see PairCfg): same roles, same arithmetic, same accumulation order.
__global__ void __cluster_dims__(2, 1, 1) __maxnreg__(PairCfg<true>::kLaunchRegs)
gemm_mxf4_pair_lite_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                           const __grid_constant__ CUtensorMap tmap_c, const ParamsP p) {
    gemm_pair_body<true>(tmap_a, tmap_b, tmap_c, p);
}

}  // namespace

cudaError_t fetch_gemm_pair_status(unsigned int* word) { return device_status_fetch(word); }

template <bool LITE, typename K>
static cudaError_t pair_kernel_init(K kernel) {
    using Cfg = PairCfg<LITE>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::kSmem);
    if (e != cudaSuccess) return e;
    // All of the SM's configurable memory as shared memory: two kernels can only share an SM under one carve-out, and
    // the small builds of GEMM and quantiser together need nearly all of it.
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, kernel);
    if (e != cudaSuccess) return e;
    if (fa.numRegs * kThreadsP < 128 * (Cfg::kRegsLight + Cfg::kRegsFwd + Cfg::kRegsEpi)) return cudaErrorLaunchOutOfResources;
    return cudaSuccess;
}

cudaError_t gemm_pair_init() {
    const cudaError_t e = pair_kernel_init<false>(gemm_mxf4_pair_kernel);
    return e != cudaSuccess ? e : pair_kernel_init<true>(gemm_mxf4_pair_lite_kernel);
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
    p.c_tma = a.has_tmap_c ? 1 : 0;
    p.accumulate = a.accumulate;
    // Tile order: groups of group_m pair-tile rows x all n-tiles.  Inside a group the A rows stay in L2 and B streams
    // through once; B is fetched from DRAM once for the whole launch only if it survives in L2 from one group to the
    // next, i.e. if a group's A rows + all of B + the group's output fit the part of L2 that behaves as one cache
    // (about half of the 126 MB: 48 MB is used here).  Eight rows where that holds, else four: on 16384 x 4096 x 16384
    // eight rows read 348 MB from DRAM, four 243 MB (operands: 168 MB) at the same speed inside a backward step;
    // groups of two or one row read a little less still but cost 0.3 % / 2.5 % of the step (fewer pairs share a B tile
    // at any moment).
    {
        const double b_bytes = (double)a.N * (double)a.K * 0.53125, out_b = a.out_fp32 ? 4.0 : 2.0;
        int gm = 8.0 * 256.0 * (double)a.K * 0.53125 + b_bytes + 8.0 * 256.0 * (double)a.N * out_b > 48.0 * 1024 * 1024 ? 4 : 8;
        const char* e = getenv("MXFP4_GEMM_GROUP_M");              // tuning switch: fixed group size (1..64) instead of the rule above
        if (e != nullptr && atoi(e) >= 1 && atoi(e) <= 64) gm = atoi(e);
        p.group_m = gm;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(kThreadsP); cfg.stream = stream;
    cfg.dynamicSmemBytes = a.lite ? PairCfg<true>::kSmem : PairCfg<false>::kSmem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, a.lite ? gemm_mxf4_pair_lite_kernel : gemm_mxf4_pair_kernel, a.tmap_a, a.tmap_b_half, a.tmap_c, p);
}

}  // namespace mx
