// Blockwise RHT + MXFP4 quantiser with the transform on the tensor cores (g in {32, 64, 128, 256}).
//
// Section 3.2 builds the blockwise RHT as a dense matrix product with a small g x g matrix, which keeps it
// memory-bound in the operand.  Here that product is a tcgen05.mma kind::f16: per tile of 128 output rows x 128
// reduce-dim elements,
//     D[128 x 128] = A[128 x 128] * T,   T = blockdiag over 128/g chunks of diag(S) H_g (x 1/sqrt(g) when exact),
// with bf16 inputs (T is +-1, +-1/8 or 0: exact) and fp32 accumulation in TMEM.  The accumulator comes back with
// one output row per TMEM lane and its 128 transformed values in consecutive columns, so each epilogue thread
// owns whole MX blocks: amax, scale, stochastic rounding and packing need no shuffles.  The same kernel serves
// both access patterns: for a contiguous reduce dimension the x tile is the K-major A operand; for the transposing
// views (W, dY^T, X^T of Algorithm 3) the very same TMA tile is handed to the MMA as an MN-major operand, so the
// transposition costs nothing.
//
// g = 256 spans two 128-wide k-tiles: H_256 = [[H_128, H_128], [H_128, -H_128]], so the two k-tiles of a 256-chunk
// go through their own half-transform T_h = diag(S_{128h..128h+127}) H_128 / 16 into two accumulators u and v, and
// the epilogue forms u + v and u - v in fp32 (one add per element more than g <= 128).
//
// One launch can quantise up to four operand views that share g, seed and rounding (the four views of one
// backward call, Algorithm 3 lines 3-6): their tiles form one list that the persistent CTAs walk, which removes
// three launch / prologue / drain gaps per layer.
//
//   warp 0        TMA producer (two 64-column x 128-row boxes per tile, 128-byte swizzle, 4-stage ring)
//   warp 1        MMA issuer (8 K=16 MMAs per tile into one of four 128-column TMEM accumulators)
//   warps 2, 3    idle: they complete warp group 0, which hands registers (setmaxnreg) to the epilogue groups
//   warps 4..19   epilogue, four groups of four warps on alternate tiles: warp = TMEM lane quadrant, a thread owns one
//                 output row of the tile: tcgen05.ld 32 columns at a time, scale / SR / pack / store per MX block
// Every mbarrier wait is bounded; on expiry the CTA records a status word and unwinds.
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx.cuh"
#include "quant_math.cuh"

namespace mx {
namespace {

constexpr int kTile = 128;                          // output rows per tile and reduce-dim elements per tile
constexpr uint32_t kBoxBytes = 64 * 2 * 128;        // one TMA box: 64 bf16 columns x 128 rows = 16 KB
constexpr uint32_t kTileBytes = 2 * kBoxBytes;      // 32 KB
constexpr uint32_t kTBytes = 2 * kBoxBytes;         // transform matrix, 128 x 128 bf16

// Two builds of the kernel.  FULL owns its SM: a 4-stage ring, four TMEM accumulators, four epilogue warp groups on
// alternate tiles.  LITE is sized to run beside the small build of the pair GEMM (gemm_pair.cu) on the same SM, so that
// the operands of one product are quantised while the other product's GEMM keeps the FP4 pipe busy: one 32 KB stage,
// one accumulator (128 TMEM columns), two epilogue warp groups that share every tile (two MX blocks of each row per
// group), 64 registers per thread at launch.  g <= 128 only.  Codes and scales are the same bytes in both builds.
template <bool LITE>
struct QCfg {
    static constexpr int kStages = LITE ? 1 : 4;
    static constexpr int kAccBufs = LITE ? 1 : 4;                        // x 128 TMEM columns
    static constexpr int kTmemCols = LITE ? 128 : 512;
    static constexpr int kEpiGroups = LITE ? 2 : 4;                      // epilogue warp groups (one warp per TMEM lane quadrant)
    static constexpr int kEpiWarps = 4 * kEpiGroups;
    static constexpr uint32_t kSmem = kStages * kTileBytes + (LITE ? 1 : 2) * kTBytes + 1024 + 256;   // FULL: two transform matrices for g = 256
    // Register hand-over (setmaxnreg): warp group 0 shrinks to kRegsLight, the epilogue groups grow to kRegsEpi.  The
    // increase can only draw on what the CTA itself holds, i.e. threads x registers-per-thread at launch: the init
    // routine checks that budget against the compiled kernel, because an increase that cannot be met waits forever.
    static constexpr int kRegsLight = LITE ? 32 : 40, kRegsEpi = LITE ? 80 : 104;
    static constexpr int kThreads = (4 + kEpiWarps) * 32;                // warp group 0: producer, MMA issuer, two idle warps; then the epilogue warp groups
    static constexpr int kLaunchRegs = LITE ? 64 : 96;
    static_assert(kThreads * kLaunchRegs >= 128 * kRegsLight + (kThreads - 128) * kRegsEpi, "warp groups ask for more registers than the CTA holds");
};

struct QView {                 // one operand view: output operand [R, K] read from x [rows, cols]
    int64_t R, K;
    uint32_t r_tiles, k_tiles;
    uint32_t tile_begin;       // first index of this view in the launch's tile list
    uint32_t n_tiles;          // r_tiles * k_tiles
    uint32_t minor_count;      // tiles along the fast direction of the view's tile order (see locate_tile)
    uint32_t d_major, d_minor; // an epilogue group's stride through the tile list, split by minor_count
    int reduce_dim;            // 1: K runs along x columns (x tile is the K-major operand); 0: along x rows (MN-major)
    uint32_t stream_tag;
    PhiloxViewConsts pv;       // index-independent part of the first three Philox rounds for this view's draws (operands < 2^36 elements)
    uint8_t* codes;
    uint8_t* scales;
    float* y_out;              // transform dump only
};

struct QParams {
    QView view[kQuantMaxViews];
    int n_views;
    uint32_t n_tiles;          // over all views
    int g, sf_native;
    const uint16_t* custom_t;  // bf16 [g, g] row-major transform matrix given by the caller, or null (then diag(S) H_g / sqrt(g))
    uint64_t seed;
    float* col_sums;           // DUAL launches: partial column sums [x rows / 128][x cols] of x in fp32 (bias gradient), or null
    PipeConsts pipe;           // see quant_math.cuh: constants kept opaque to the compiler
    PhiloxKeys keys;           // the ten Philox round keys of `seed` (key schedule only; the rounds run on the device)
};

struct QMaps {
    CUtensorMap x[kQuantMaxViews];
};

// Position of a tile in the launch's list: its view and its (row tile, k tile) there.  Tiles of a view with a
// contiguous reduce dimension run along k first, the transposing ones along the output rows first, so that CTAs
// working side by side read neighbouring 256-byte row segments of x.
struct TilePos {
    int v;
    uint32_t rt, kt;
    uint32_t local;            // index inside the view
};
__device__ __forceinline__ TilePos locate_tile(const QParams& p, uint32_t t) {
    int v = 0;
#pragma unroll
    for (int i = 1; i < kQuantMaxViews; ++i)
        if (i < p.n_views && t >= p.view[i].tile_begin) v = i;
    const uint32_t local = t - p.view[v].tile_begin;
    TilePos pos;
    pos.v = v;
    pos.local = local;
    if (p.view[v].reduce_dim == 1) { pos.rt = local / p.view[v].k_tiles; pos.kt = local - pos.rt * p.view[v].k_tiles; }
    else { pos.kt = local / p.view[v].r_tiles; pos.rt = local - pos.kt * p.view[v].r_tiles; }
    return pos;
}
// The position `stride` tiles further on (stride = the view's d_major * minor_count + d_minor): additions only while
// the walk stays inside the view.
__device__ __forceinline__ TilePos advance_tile(const QParams& p, const TilePos& cur, uint32_t t_next) {
    const QView& vw = p.view[cur.v];
    TilePos pos = cur;
    pos.local = cur.local + vw.d_major * vw.minor_count + vw.d_minor;
    if (pos.local >= vw.n_tiles) return locate_tile(p, t_next);
    uint32_t major = (vw.reduce_dim == 1 ? cur.rt : cur.kt) + vw.d_major, minor = (vw.reduce_dim == 1 ? cur.kt : cur.rt) + vw.d_minor;
    if (minor >= vw.minor_count) { minor -= vw.minor_count; ++major; }
    if (vw.reduce_dim == 1) { pos.rt = major; pos.kt = minor; } else { pos.kt = major; pos.rt = minor; }
    return pos;
}

// DUAL launches: view 0 (reduce along x columns) and view 1 (reduce along x rows) are the two views of ONE tensor x
// (dY of Algorithm 3, lines 3 and 5).  A unit is one 128 x 128 tile of x, loaded once; it yields two logical tiles,
// 2 u (view 0: rows = x rows) and 2 u + 1 (view 1: rows = x columns).  Units run along x columns first.
__device__ __forceinline__ TilePos locate_dual(const QParams& p, uint32_t t) {
    const uint32_t u = t >> 1, xc_tiles = p.view[0].k_tiles;
    const uint32_t xr = u / xc_tiles, xc = u - xr * xc_tiles;
    TilePos pos;
    pos.v = (int)(t & 1u);
    pos.local = u;
    if (pos.v == 0) { pos.rt = xr; pos.kt = xc; } else { pos.rt = xc; pos.kt = xr; }
    return pos;
}

enum { kModeSR = 0, kModeRN = 1, kModeDump = 2, kModeSR16 = 3 };
constexpr bool mode_draws(int mode) { return mode == kModeSR || mode == kModeSR16; }
// template argument of quantize_block32_rw; the g = 256 kernel (kw = 2) rounds SR through the convert instruction (same codes, fewer registers)
constexpr int mode_rounding(int mode, int kw) { return mode == kModeSR16 ? 2 : (mode == kModeSR && kw == 2) ? 3 : mode; }

// The 32 draws of a block.  FOLD: with the view's precomputed constants (fewer instructions, five more live values: pays
// where registers are not the limit, i.e. in the SR16 kernel; the integer SR path and the g = 256 kernel lose with it).
template <bool FOLD>
__device__ __forceinline__ void view_draws32(const PhiloxKeys& ks, uint32_t stream_tag, const PhiloxViewConsts* pv, uint64_t i0, uint32_t (&rw)[8]) {
    if (FOLD) sr_draws32_view(ks, *pv, i0, rw);
    else sr_draws32(ks, stream_tag, i0, rw);
}

// KW = 128-wide k-tiles per entry of the tile list: 1, or 2 for g = 256 (a tile then spans one 256-chunk).
template <int MODE, int KW, bool LITE, bool DUAL>
__device__ __forceinline__ void quantize_tc_body(const QMaps& maps, const QParams& p) {
    using Cfg = QCfg<LITE>;
    static_assert(!DUAL || (KW == 1 && !LITE), "one load for two views: g <= 128, full-size build");
    constexpr int kStagesQ = Cfg::kStages, kAccBufs = Cfg::kAccBufs, kEpiGroups = Cfg::kEpiGroups, kThreadsQ = Cfg::kThreads;
    static_assert(!(LITE && KW == 2), "the small build serves g <= 128");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* smem_t = smem + kStagesQ * kTileBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_t + (LITE ? 1 : 2) * kTBytes);
    uint64_t* full_bar = bars;                          // [kStagesQ]  TMA -> MMA
    uint64_t* empty_bar = bars + kStagesQ;              // [kStagesQ]  MMA -> TMA
    uint64_t* acc_full = bars + 2 * kStagesQ;           // [kAccBufs]  MMA -> epilogue
    uint64_t* acc_empty = bars + 2 * kStagesQ + kAccBufs;   // [kAccBufs]  epilogue -> MMA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStagesQ + 2 * kAccBufs);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t num_tiles = p.n_tiles;
    constexpr bool kFold = MODE == kModeSR16 && KW == 1;

    if (threadIdx.x == 0) {
        // a stage is free when its transforms have read it (one commit) and, with column sums on, the two summing warps too
        const uint32_t n_readers = (DUAL && p.col_sums != nullptr) ? 3u : 1u;
        for (int s = 0; s < kStagesQ; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], n_readers); }
        for (int b = 0; b < kAccBufs; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], (KW == 2 || LITE) ? 8 : 4); }
        *abort_flag = 0;
        mbar_fence_init();
        for (int v = 0; v < p.n_views; ++v) prefetch_tensormap(&maps.x[v]);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, Cfg::kTmemCols);
        tmem_relinquish();
    }
    {
        if (KW == 1 && p.custom_t != nullptr) pdl_wait();                // the matrix may come from the kernel before this one
        // Transform operand, written in the 128-byte-swizzled K-major layout the MMA descriptor expects:
        // entry (n, k) at box (k / 64), row n (128 B pitch), 16-byte chunk ((k % 64) / 8) ^ (n % 8).
#pragma unroll
        for (int h = 0; h < KW; ++h) {                                   // KW = 2: sign bits 128 h .. 128 h + 127 come from Philox call h
            const uint4 o = philox4x32_10((uint32_t)h, 0u, 0u, 0u, (uint32_t)p.seed, (uint32_t)(p.seed >> 32));
            const uint32_t sign[4] = {o.x, o.y, o.z, o.w};
            for (int task = threadIdx.x; task < 128 * 16; task += kThreadsQ) {
                const int n = task >> 4, c = task & 15;                  // c: 16-byte chunk = 8 consecutive k
                uint32_t w[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int k0 = c * 8 + 2 * j;
                    if (KW == 1 && p.custom_t != nullptr) {
                        // entry (n, k) of the operand = T[k % g][n % g] inside a g-chunk, 0 across chunks (Section 3.2: any orthogonal matrix)
                        const int gm = p.g - 1;
                        const bool same = ((n ^ k0) & ~gm) == 0;              // k0 and k0 + 1 lie in the same chunk (g is even)
                        const uint32_t lo = same ? p.custom_t[(k0 & gm) * p.g + (n & gm)] : 0u;
                        const uint32_t hi = same ? p.custom_t[((k0 + 1) & gm) * p.g + (n & gm)] : 0u;
                        w[j] = lo | (hi << 16);
                    } else {
                        w[j] = KW == 2 ? (transform_entry_256(n, k0, sign) | (transform_entry_256(n, k0 + 1, sign) << 16))
                                       : (transform_entry(n, k0, p.g, sign) | (transform_entry(n, k0 + 1, p.g, sign) << 16));
                    }
                }
                const uint32_t off = (uint32_t)(c >> 3) * kBoxBytes + (uint32_t)n * 128u + (uint32_t)(((c & 7) ^ (n & 7)) << 4);
                *reinterpret_cast<uint4*>(smem_t + h * kTBytes + off) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
        fence_proxy_async_smem();                                        // generic-proxy writes -> tensor-core reads
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    pdl_launch_dependents();                            // the next kernel of the stream may set itself up behind this one
    pdl_wait();                                         // the set-up above overlapped the previous kernel's tail; its data is needed now

    if (warp < 4) {
    // ============================ warp group 0: producer, MMA issuer, two idle warps; it gives registers to the others
    reg_dealloc<Cfg::kRegsLight>();
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            // DUAL: one load per unit (two logical tiles), in the coordinates of its row-wise view
            for (uint32_t t = DUAL ? 2u * blockIdx.x : blockIdx.x; t < num_tiles && ok; t += (DUAL ? 2u : 1u) * gridDim.x) {
                const TilePos pos = DUAL ? locate_dual(p, t) : locate_tile(p, t);
                // x coordinates: (column, row).  reduce_dim 1: output rows = x rows, k = x columns; else swapped.
                const bool rowwise = p.view[pos.v].reduce_dim == 1;
#pragma unroll
                for (int h = 0; h < KW; ++h, ++it) {
                    const int s = it % kStagesQ;
                    if (!(ok = mbar_wait(&empty_bar[s], ((it / kStagesQ) & 1) ^ 1, abort_flag))) break;
                    const uint32_t kt = pos.kt * KW + h;                 // 128-wide k-tile
                    const int32_t cx = (int32_t)((rowwise ? kt : pos.rt) * kTile), cy = (int32_t)((rowwise ? pos.rt : kt) * kTile);
                    uint8_t* st = smem + s * kTileBytes;
                    mbar_expect_tx(&full_bar[s], kTileBytes);
                    tma_load_2d(st, &maps.x[pos.v], &full_bar[s], cx, cy);
                    tma_load_2d(st + kBoxBytes, &maps.x[pos.v], &full_bar[s], cx + 64, cy);
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // kind::f16 instruction descriptor: D = fp32 (bits 4-5 = 1), A = B = bf16 (bits 7-9, 10-12 = 1),
            // A major at bit 15 (0 = K-major, 1 = MN-major), B K-major, N >> 3 at bit 17, M >> 4 at bit 24.
            const uint32_t idesc_k = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTile >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);
            const uint32_t t_addr = smem_u32(smem_t);
            uint32_t it = 0;
            bool ok = true;
            auto transform = [&](uint32_t a_addr, bool rowwise, int h, int b) {      // 8 MMAs: stage -> accumulator b
                const uint32_t idesc = idesc_k | ((rowwise ? 0u : 1u) << 15);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {                           // K = 16 per MMA
                    uint64_t adesc;
                    if (rowwise)            // K-major: box ks/4, 32 bytes of K per step inside the 128-byte swizzle atom
                        adesc = make_smem_desc(a_addr + (ks >> 2) * kBoxBytes + (ks & 3) * 32, 16, 1024, 2);
                    else                    // MN-major: 16 k-rows of 128 B per step; the second 64 output rows sit one box further
                        adesc = make_smem_desc(a_addr + ks * 2048, kBoxBytes, 1024, 2);
                    const uint64_t bdesc = make_smem_desc(t_addr + h * kTBytes + (ks >> 2) * kBoxBytes + (ks & 3) * 32, 16, 1024, 2);
                    tc_mma_f16(tmem_base + b * kTile, adesc, bdesc, idesc, ks != 0 ? 1u : 0u);
                }
            };
            if (DUAL) {
                // per unit: the stage is the K-major operand of view 0's transform and the MN-major operand of view 1's
                uint32_t is = 0;                                             // stage counter (units)
                for (uint32_t u = blockIdx.x; 2u * u < num_tiles && ok; u += gridDim.x, ++is) {
                    const int s = is % kStagesQ;
                    if (!(ok = mbar_wait(&full_bar[s], (is / kStagesQ) & 1, abort_flag))) break;
                    const uint32_t a_addr = smem_u32(smem + s * kTileBytes);
                    for (int h = 0; h < 2 && ok; ++h, ++it) {
                        const int b = it % kAccBufs;
                        if (!(ok = mbar_wait(&acc_empty[b], ((it / kAccBufs) & 1) ^ 1, abort_flag))) break;
                        tc_fence_after_sync();
                        transform(a_addr, h == 0, 0, b);
                        tc_commit(&acc_full[b]);
                    }
                    if (ok) tc_commit(&empty_bar[s]);                        // both transforms have read the stage
                }
            } else
            for (uint32_t t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
                int v = 0;
#pragma unroll
                for (int i = 1; i < kQuantMaxViews; ++i)
                    if (i < p.n_views && t >= p.view[i].tile_begin) v = i;
                const bool rowwise = p.view[v].reduce_dim == 1;
#pragma unroll
                for (int h = 0; h < KW; ++h, ++it) {                       // KW = 2: k-tile h goes through T_h into its own accumulator
                    const int s = it % kStagesQ, b = it % kAccBufs;
                    if (!(ok = mbar_wait(&acc_empty[b], ((it / kAccBufs) & 1) ^ 1, abort_flag))) break;
                    if (!(ok = mbar_wait(&full_bar[s], (it / kStagesQ) & 1, abort_flag))) break;
                    tc_fence_after_sync();
                    transform(smem_u32(smem + s * kTileBytes), rowwise, h, b);
                    tc_commit(&empty_bar[s]);
                    tc_commit(&acc_full[b]);
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (DUAL && p.col_sums != nullptr) {
        // ------------------------------------------------------------------ warps 2, 3: column sums of the x tile (dL/db = 1 dL/dy)
        // The tile is in shared memory anyway: warp w sums columns 64 w .. 64 w + 63 (one TMA box), a lane two adjacent
        // columns (one 32-bit word per row; the 128-byte swizzle permutes 16-byte chunks inside a row, so a warp's 32
        // words of a row still fall into 32 different banks), rows in order: a fixed summation order.  One partial sum
        // per (128-row band of x, column); a second kernel adds the bands in order.
        const int w = warp - 2;
        uint32_t is = 0;
        bool ok = true;
        for (uint32_t u = blockIdx.x; 2u * u < num_tiles; u += gridDim.x, ++is) {
            const int s = is % kStagesQ;
            ok = mbar_wait(&full_bar[s], (is / kStagesQ) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint8_t* box = smem + s * kTileBytes + w * kBoxBytes;
            float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
            for (int r = 0; r < kTile; ++r) {
                const uint32_t v = *reinterpret_cast<const uint32_t*>(box + r * 128 + ((((lane >> 2) ^ (r & 7)) << 4) | ((lane & 3) << 2)));
                s0 += __uint_as_float(v << 16);
                s1 += __uint_as_float(v & 0xFFFF0000u);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[s]);                   // this warp is done with the stage
            const uint32_t xc_tiles = p.view[0].k_tiles, xr = u / xc_tiles, xc = u - xr * xc_tiles;
            float* dst = p.col_sums + (int64_t)xr * p.view[0].K + (int64_t)xc * kTile + w * 64 + 2 * lane;
            *reinterpret_cast<float2*>(dst) = make_float2(s0, s1);
        }
        if (!ok && lane == 0) *abort_flag = 1;
    }
    } else {
        // ------------------------------------------------------------------ epilogue (warp groups 1..4)
        reg_alloc<Cfg::kRegsEpi>();
        // Four groups of four warps take alternate tiles; inside a group a warp owns one TMEM lane quadrant, i.e. a
        // thread owns one output row of the tile: four MX blocks, 64 bytes of codes, 4 scale bytes.  The SR draws of a
        // block are computed while the block before it is rounded (for a tile's first block: at the end of the tile
        // before); they depend only on element indices.
        const int e = warp - 4;
        const int q = warp & 3;                      // TMEM lane quadrant this warp may read
        const int grp = e >> 2;
        const float cg = p.custom_t != nullptr ? 1.0f : p.g == 32 ? 0.17677669529663687f : p.g == 128 ? 0.08838834764831845f : 1.0f;
        // FULL: the groups take alternate tiles.  LITE: both groups take every tile of the CTA, group 0 the row's MX
        // blocks 0 and 1, group 1 blocks 2 and 3.
        const uint32_t stride = (LITE ? 1u : (uint32_t)kEpiGroups) * gridDim.x;
        constexpr int kBlocksPerThread = LITE ? 2 : 4;
        const int jb = LITE ? 2 * grp : 0;                          // first MX block of the row this thread handles
        const uint32_t lane_row = (uint32_t)(q * 32 + lane);
        bool ok = true;

        auto first_elem = [&](const TilePos& pos) -> uint64_t {          // linear index of this thread's first element
            return (uint64_t)(pos.rt * (uint32_t)kTile + lane_row) * (uint64_t)p.view[pos.v].K + (uint64_t)(pos.kt * (uint32_t)(kTile * KW));
        };

        // logical tile of this CTA's i-th accumulator: tiles are dealt out round-robin; in a DUAL launch whole units are
        // (two consecutive logical tiles, one per view), so that both transforms of a unit read the same stage
        auto tile_of = [&](uint32_t i) -> uint32_t {
            return DUAL ? 2u * (blockIdx.x + (i >> 1) * gridDim.x) + (i & 1u) : blockIdx.x + i * gridDim.x;
        };
        uint32_t it = LITE ? 0u : (uint32_t)grp;
        uint32_t t = tile_of(it);
        TilePos pos = DUAL ? locate_dual(p, t < num_tiles ? t : 0u) : locate_tile(p, t < num_tiles ? t : 0u);
        uint32_t rw[8];
        if (mode_draws(MODE)) view_draws32<kFold>(p.keys, p.view[pos.v].stream_tag, &p.view[pos.v].pv, first_elem(pos) + 32u * jb, rw);
        if (KW == 2) {
            // g = 256: a tile is one 256-chunk of 128 rows; its two k-tiles went through T_0 and T_1 into the accumulator
            // pair (b0, b0 + 1): u = A_lo T_0, v = A_hi T_1.  The transformed values are y[0..127] = u + v and
            // y[128..255] = u - v (H_256 = [[H, H], [H, -H]]).  Tiles alternate between the two accumulator pairs; pair
            // pr is drained by groups 2 pr (the u + v half) and 2 pr + 1 (the u - v half), so every barrier is used by
            // the same warps each time and its phases alternate for them.
            const int pr = grp >> 1, hh = grp & 1;
            const uint32_t stride2 = 2u * gridDim.x;
            it = (uint32_t)pr;
            t = blockIdx.x + it * gridDim.x;
            pos = locate_tile(p, t < num_tiles ? t : 0u);
            if (mode_draws(MODE)) view_draws32<kFold>(p.keys, p.view[pos.v].stream_tag, &p.view[pos.v].pv, first_elem(pos) + 128u * hh, rw);
            for (; t < num_tiles; t += stride2, it += 2) {
                const int b0 = 2 * pr;
                const QView& vw = p.view[pos.v];
                const uint32_t rt = pos.rt, kt = pos.kt;
                const int64_t K = vw.K;
                const int64_t row = (int64_t)rt * kTile + lane_row;
                const int64_t k0 = (int64_t)kt * (2 * kTile) + 128 * hh;        // this group's 128 elements of the row
                const bool live = row < vw.R;
                uint8_t* code_dst = vw.codes + row * (K >> 1) + (k0 >> 1);
                const uint32_t nkb = (uint32_t)(K >> 5), nkc = (nkb + 3) >> 2;
                uint8_t* scale_dst = vw.scales + (p.sf_native ? ((int64_t)(rt * nkc + 2 * kt + hh) * 512 + lane * 16 + q * 4) : row * nkb + (k0 >> 5));
                float* y_dst = MODE == kModeDump ? vw.y_out + row * K + k0 : nullptr;
                const uint64_t i_cur = first_elem(pos) + 128u * hh;
                const uint32_t tag_cur = vw.stream_tag;
                const PhiloxViewConsts* pv_cur = &vw.pv;
                pos = t + stride2 < num_tiles ? advance_tile(p, pos, t + stride2) : locate_tile(p, 0u);
                const uint64_t i_next = first_elem(pos) + 128u * hh;
                const uint32_t tag_next = p.view[pos.v].stream_tag;
            const PhiloxViewConsts* pv_next = &p.view[pos.v].pv;
                const uint32_t ph = (it >> 1) & 1;                               // this pair's (it / 2)-th use
                ok = mbar_wait(&acc_full[b0], ph, abort_flag) && mbar_wait(&acc_full[b0 + 1], ph, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t ta = tmem_base + ((uint32_t)(q * 32) << 16) + b0 * kTile;
                uint32_t sb_all = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t nx[8], packed[4], sb = 0;
                    float y[32];
#pragma unroll
                    for (int c = 0; c < 2; ++c) {                           // sixteen columns of u and of v at a time
                        uint32_t u[16], v[16];
                        tmem_ld_32x32b_x16(ta + 32 * j + 16 * c, u);
                        tmem_ld_32x32b_x16(ta + kTile + 32 * j + 16 * c, v);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            y[16 * c + i] = hh == 0 ? __uint_as_float(u[i]) + __uint_as_float(v[i]) : __uint_as_float(u[i]) - __uint_as_float(v[i]);
                    }
                    if (j == 3) {                                           // this group is done with both accumulators
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) { mbar_arrive(&acc_empty[b0]); mbar_arrive(&acc_empty[b0 + 1]); }
                    }
                    if (mode_draws(MODE)) {
                        if (j < 3) view_draws32<kFold>(p.keys, tag_cur, pv_cur, i_cur + 32 * (j + 1), nx);
                        else view_draws32<kFold>(p.keys, tag_next, pv_next, i_next, nx);
                    }
                    if (MODE == kModeDump) {
                        if (live) {
                            float4* dst = reinterpret_cast<float4*>(y_dst + 32 * j);
#pragma unroll
                            for (int i = 0; i < 8; ++i) dst[i] = make_float4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
                        }
                    } else {
                        quantize_block32_rw<mode_rounding(MODE, KW)>(y, rw, packed, sb, p.pipe);
                        if (live) *reinterpret_cast<uint4*>(code_dst + 16 * j) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                        sb_all |= sb << (8 * j);
                    }
                    if (mode_draws(MODE)) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) rw[i] = nx[i];
                    }
                }
                if (MODE != kModeDump && live) *reinterpret_cast<uint32_t*>(scale_dst) = sb_all;
            }
        } else
        for (; t < num_tiles; it += (LITE ? 1 : kEpiGroups), t = DUAL ? tile_of(it) : t + stride) {
            const int b = it % kAccBufs;
            const QView& vw = p.view[pos.v];
            const uint32_t rt = pos.rt, kt = pos.kt;
            const int64_t K = vw.K;
            const int64_t row = (int64_t)rt * kTile + lane_row;                 // output row
            const int64_t k0 = (int64_t)kt * kTile;
            const bool live = row < vw.R;
            uint8_t* code_dst = vw.codes + row * (K >> 1) + (k0 >> 1);
            const uint32_t nkb = (uint32_t)(K >> 5), nkc = (nkb + 3) >> 2;
            uint8_t* scale_dst = vw.scales + (p.sf_native ? ((int64_t)(rt * nkc + kt) * 512 + lane * 16 + q * 4) : row * nkb + (k0 >> 5));
            float* y_dst = MODE == kModeDump ? vw.y_out + row * K + k0 : nullptr;
            const uint64_t i_cur = first_elem(pos);
            const uint32_t tag_cur = vw.stream_tag;
            const PhiloxViewConsts* pv_cur = &vw.pv;
            // position of the next tile of this group (past the end: computed but not used)
            if (DUAL) {
                const uint32_t t_next = tile_of(it + kEpiGroups);
                pos = locate_dual(p, t_next < num_tiles ? t_next : 0u);
            } else {
                pos = t + stride < num_tiles ? advance_tile(p, pos, t + stride) : locate_tile(p, 0u);
            }
            const uint64_t i_next = first_elem(pos);
            const uint32_t tag_next = p.view[pos.v].stream_tag;
            const PhiloxViewConsts* pv_next = &p.view[pos.v].pv;
            ok = mbar_wait(&acc_full[b], (it / kAccBufs) & 1, abort_flag);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + b * kTile;
            uint32_t sb_all = 0;
#pragma unroll
            for (int jj = 0; jj < kBlocksPerThread; ++jj) {
                const int j = jb + jj;                          // MX block of the row
                uint32_t raw[32], nx[8], packed[4], sb = 0;
                float y[32];
                tmem_ld_32x32b_x32(taddr + 32 * j, raw);
                tmem_ld_wait();
                if (jj == kBlocksPerThread - 1) {               // the accumulator is free once it has been read
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[b]);
                }
                if (mode_draws(MODE)) {
                    if (jj < kBlocksPerThread - 1) view_draws32<kFold>(p.keys, tag_cur, pv_cur, i_cur + 32 * (j + 1), nx);
                    else view_draws32<kFold>(p.keys, tag_next, pv_next, i_next + 32u * jb, nx);
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) y[i] = __uint_as_float(raw[i]);
                if (cg != 1.0f) {                               // g = 32, 128: 1/sqrt(g) is not a power of two (for g = 64 it is folded into T)
#pragma unroll
                    for (int i = 0; i < 32; ++i) y[i] *= cg;
                }
                if (MODE == kModeDump) {
                    if (live) {
                        float4* dst = reinterpret_cast<float4*>(y_dst + 32 * j);
#pragma unroll
                        for (int i = 0; i < 8; ++i) dst[i] = make_float4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
                    }
                } else {
                    quantize_block32_rw<mode_rounding(MODE, KW)>(y, rw, packed, sb, p.pipe);
                    if (live) *reinterpret_cast<uint4*>(code_dst + 16 * j) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    sb_all |= sb << (8 * jj);
                }
                if (mode_draws(MODE)) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) rw[i] = nx[i];
                }
            }
            if (MODE != kModeDump && live) {
                if (LITE) *reinterpret_cast<uint16_t*>(scale_dst + jb) = (uint16_t)sb_all;   // this group's two of the row's four scale bytes
                else *reinterpret_cast<uint32_t*>(scale_dst) = sb_all;                     // four consecutive bytes in either scale layout
            }
        }
        if (!ok && lane == 0) *abort_flag = 1;
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, Cfg::kTmemCols);
    }
}

template <int MODE, int KW>
__global__ void __launch_bounds__(QCfg<false>::kThreads, 1)
quantize_tc_kernel(const __grid_constant__ QMaps maps, const __grid_constant__ QParams p) {
    quantize_tc_body<MODE, KW, false, false>(maps, p);
}

// Both views of one tensor from one read of it (Algorithm 3 lines 3 and 5 use the same dL/dy), g <= 128.
template <int MODE>
__global__ void __launch_bounds__(QCfg<false>::kThreads, 1)
quantize_tc_dual_kernel(const __grid_constant__ QMaps maps, const __grid_constant__ QParams p) {
    quantize_tc_body<MODE, 1, false, true>(maps, p);
}

// The small-footprint build (see QCfg), g <= 128.
template <int MODE>
__global__ void __maxnreg__(QCfg<true>::kLaunchRegs)
quantize_tc_lite_kernel(const __grid_constant__ QMaps maps, const __grid_constant__ QParams p) {
    quantize_tc_body<MODE, 1, true, false>(maps, p);
}

}  // namespace

bool quant_tc_eligible(const QuantArgs& a) {
    const int64_t K = a.reduce_dim == 1 ? a.cols : a.rows;
    const int64_t R = a.reduce_dim == 1 ? a.rows : a.cols;
    const int64_t tiles = ((R + kTile - 1) / kTile) * (K / kTile);          // tile indices are 32-bit in the kernel
    // the element index that keys the SR draws stays below 2^36 (the kernel folds a zero high counter word into its constants)
    return (a.g == 32 || a.g == 64 || a.g == 128 || a.g == 256) && K % kTile == 0 && tiles < (int64_t(1) << 28) && a.has_tmap &&
           R * K < (int64_t(1) << 36);
}

cudaError_t fetch_quant_tc_status(unsigned int* word) { return device_status_fetch(word); }

template <bool LITE>
static cudaError_t quant_kernel_init(const void* k) {
    using Cfg = QCfg<LITE>;
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg::kSmem);
    if (e != cudaSuccess) return e;
    // all of the SM's configurable memory as shared memory (see gemm_pair.cu: kernels share an SM only under one carve-out)
    e = cudaFuncSetAttribute(k, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, k);
    if (e != cudaSuccess) return e;
    // registers the CTA holds at launch must cover the limits the warp groups set for themselves
    if (fa.numRegs * Cfg::kThreads < 128 * Cfg::kRegsLight + (Cfg::kThreads - 128) * Cfg::kRegsEpi) return cudaErrorLaunchOutOfResources;
    return cudaSuccess;
}

cudaError_t quant_tc_init() {
    const void* kernels[8] = {(const void*)quantize_tc_kernel<kModeSR, 1>, (const void*)quantize_tc_kernel<kModeRN, 1>,
                              (const void*)quantize_tc_kernel<kModeDump, 1>, (const void*)quantize_tc_kernel<kModeSR16, 1>,
                              (const void*)quantize_tc_kernel<kModeSR, 2>, (const void*)quantize_tc_kernel<kModeRN, 2>,
                              (const void*)quantize_tc_kernel<kModeDump, 2>, (const void*)quantize_tc_kernel<kModeSR16, 2>};
    for (const void* k : kernels) {
        const cudaError_t e = quant_kernel_init<false>(k);
        if (e != cudaSuccess) return e;
    }
    const void* dual[3] = {(const void*)quantize_tc_dual_kernel<kModeSR>, (const void*)quantize_tc_dual_kernel<kModeRN>,
                           (const void*)quantize_tc_dual_kernel<kModeSR16>};
    for (const void* k : dual) {
        const cudaError_t e = quant_kernel_init<false>(k);
        if (e != cudaSuccess) return e;
    }
    const void* lite[3] = {(const void*)quantize_tc_lite_kernel<kModeSR>, (const void*)quantize_tc_lite_kernel<kModeRN>,
                           (const void*)quantize_tc_lite_kernel<kModeSR16>};
    for (const void* k : lite) {
        const cudaError_t e = quant_kernel_init<true>(k);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// Quantise n (1..kQuantMaxViews) eligible operand views that share g, seed, rounding and scale layout in one launch.
cudaError_t launch_quantize_tc_group(const QuantArgs* a, int n, bool dump_y, cudaStream_t stream, bool lite, bool dual, float* col_sums) {
    if (n < 1 || n > kQuantMaxViews) return cudaErrorInvalidValue;
    // dual: a[0] and a[1] are the row-wise and the transposed view of one tensor, whose tiles are then loaded once for both
    if (dual && (n != 2 || lite || dump_y || a[0].g == 256 || a[0].custom_t != nullptr || a[0].x != a[1].x || a[0].rows != a[1].rows ||
                 a[0].cols != a[1].cols || a[0].ld != a[1].ld || a[0].reduce_dim != 1 || a[1].reduce_dim != 0 || a[0].rows % kTile != 0))
        return cudaErrorInvalidValue;
    if (lite && (dump_y || a[0].g == 256 || a[0].custom_t != nullptr)) return cudaErrorInvalidValue;   // the small build: RHT with g <= 128, quantising
    QParams p;
    QMaps maps;
    uint32_t tiles = 0;
    for (int v = 0; v < n; ++v) {
        QView& w = p.view[v];
        w.R = a[v].reduce_dim == 1 ? a[v].rows : a[v].cols;
        w.K = a[v].reduce_dim == 1 ? a[v].cols : a[v].rows;
        w.r_tiles = (uint32_t)((w.R + kTile - 1) / kTile);
        w.k_tiles = (uint32_t)(w.K / (a[v].g == 256 ? 2 * kTile : kTile));     // g = 256: a tile spans one 256-chunk
        w.tile_begin = tiles;
        w.n_tiles = w.r_tiles * w.k_tiles;
        tiles += w.n_tiles;
        w.reduce_dim = a[v].reduce_dim;
        w.stream_tag = a[v].stream_tag;
        w.codes = a[v].codes; w.scales = a[v].scales; w.y_out = a[v].y_out;
        maps.x[v] = a[v].tmap_x;
    }
    for (int v = n; v < kQuantMaxViews; ++v) { p.view[v] = p.view[0]; p.view[v].tile_begin = 0xFFFFFFFFu; maps.x[v] = maps.x[0]; }
    p.n_views = n;
    p.n_tiles = tiles;
    p.g = a[0].g; p.sf_native = a[0].sf_native; p.seed = a[0].seed;
    p.custom_t = static_cast<const uint16_t*>(a[0].custom_t);
    if (p.custom_t != nullptr && p.g == 256) return cudaErrorInvalidValue;
    if (col_sums != nullptr && !dual) return cudaErrorInvalidValue;
    p.col_sums = col_sums;
    p.pipe = make_pipe_consts();
    {   // Philox key schedule: key_i = key_0 + i * (0x9E3779B9, 0xBB67AE85)
        uint32_t k0 = (uint32_t)p.seed, k1 = (uint32_t)(p.seed >> 32);
        for (int i = 0; i < 10; ++i) {
            p.keys.k0[i] = k0; p.keys.k1[i] = k1;
            k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
        }
    }
    for (int v = 0; v < kQuantMaxViews; ++v) p.view[v].pv = philox_view_consts(p.keys, p.view[v].stream_tag);
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const uint32_t units = dual ? tiles / 2 : tiles;       // loads: in a dual launch the two views' tiles pair up
    const unsigned grid = units < (uint32_t)sms ? units : (unsigned)sms;
    for (int v = 0; v < kQuantMaxViews; ++v) {
        QView& w = p.view[v];
        w.minor_count = w.reduce_dim == 1 ? w.k_tiles : w.r_tiles;
        // tiles between two visits of an epilogue group: the groups take alternate tiles (g = 256: in pairs; small build: every tile)
        const uint32_t step = (lite ? 1u : p.g == 256 ? 2u : (uint32_t)QCfg<false>::kEpiGroups) * grid;
        w.d_major = step / w.minor_count;
        w.d_minor = step % w.minor_count;
    }
    const bool wide = p.g == 256;
    void (*kernel)(QMaps, QParams);
    if (dual) kernel = a[0].rounding == 0 ? quantize_tc_dual_kernel<kModeSR> : a[0].rounding == 2 ? quantize_tc_dual_kernel<kModeSR16> : quantize_tc_dual_kernel<kModeRN>;
    else if (lite) kernel = a[0].rounding == 0 ? quantize_tc_lite_kernel<kModeSR> : a[0].rounding == 2 ? quantize_tc_lite_kernel<kModeSR16> : quantize_tc_lite_kernel<kModeRN>;
    else if (dump_y) kernel = wide ? quantize_tc_kernel<kModeDump, 2> : quantize_tc_kernel<kModeDump, 1>;
    else if (a[0].rounding == 0) kernel = wide ? quantize_tc_kernel<kModeSR, 2> : quantize_tc_kernel<kModeSR, 1>;
    else if (a[0].rounding == 2) kernel = wide ? quantize_tc_kernel<kModeSR16, 2> : quantize_tc_kernel<kModeSR16, 1>;
    else kernel = wide ? quantize_tc_kernel<kModeRN, 2> : quantize_tc_kernel<kModeRN, 1>;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.stream = stream;
    cfg.blockDim = dim3(lite ? QCfg<true>::kThreads : QCfg<false>::kThreads);
    cfg.dynamicSmemBytes = lite ? QCfg<true>::kSmem : QCfg<false>::kSmem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, maps, p);
}

cudaError_t launch_quantize_tc(const QuantArgs& a, bool dump_y, cudaStream_t stream) {
    return launch_quantize_tc_group(&a, 1, dump_y, stream, false, false, nullptr);
}

}  // namespace mx
