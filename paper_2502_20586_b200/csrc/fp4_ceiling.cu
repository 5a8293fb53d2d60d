// On-box ceiling of the block-scaled FP4 tensor pipe: every CTA pair issues back-to-back
// tcgen05.mma.cta_group::2.kind::mxf4.block_scale (256 x 256 x 64 per instruction) on operands that are already
// resident in shared memory (pseudo-random E2M1 codes, all scales 1.0), with no loads and no epilogue.  The rate it
// reaches is what a GEMM could reach if nothing but the tensor pipe limited it; bench.py times it with CUDA events
// and prints it beside the nominal and the bf16-derived peaks.  Not part of the method; no output is produced.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/mxfp4.h"
#include "kernels.h"
#include "ptx.cuh"

namespace mx {
namespace {

constexpr int kStagesC = 4;                              // operand sets the MMAs rotate through
constexpr uint32_t kTileC = 128 * 128;                   // 128 rows x 128 B (256 E2M1 elements of K)
constexpr uint32_t kSmemC = kStagesC * 2 * kTileC + 1024 + 64;
constexpr int kBatch = 32;                               // MMAs per commit
constexpr int kThreadsC = 5 * 32;                        // warp 0: issuer; warps 1..4: one per TMEM lane quadrant (scale fill)

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreadsC, 1)
fp4_ceiling_kernel(uint32_t batches) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStagesC * 2 * kTileC);     // [2] batch complete (ping-pong)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();

    if (threadIdx.x == 0) {
        mbar_init(&bars[0], 1);
        mbar_init(&bars[1], 1);
        mbar_fence_init();
    }
    // operands: a multiplicative hash of the byte index, different per CTA
    for (uint32_t i = threadIdx.x; i < kStagesC * 2 * kTileC / 4; i += kThreadsC)
        reinterpret_cast<uint32_t*>(smem)[i] = (i * 4u + blockIdx.x * 0x9E3779B9u + 1u) * 0x85EBCA6Bu ^ ((i + 7u) * 0xC2B2AE35u >> 7);
    fence_proxy_async_smem();
    if (warp == 0) {
        tmem_alloc_pair(tmem_slot, 512);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp >= 1) {                                     // scales: byte 127 = 2^0 in every column the MMAs read
        const uint32_t lane_base = (uint32_t)(((warp - 1) & 3) * 32) << 16;
        const uint4 ones = make_uint4(0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu, 0x7F7F7F7Fu);
        tmem_st_32x32b_x8(tmem_base + lane_base + 256, ones, ones);
        tmem_st_32x32b_x16(tmem_base + lane_base + 264, ones, ones, ones, ones);
        tmem_st_wait();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after_sync();

    if (warp == 0 && lane == 0 && rank == 0) {
        const uint32_t idesc0 = (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | (1u << 23) | ((256u >> 4) << 24);
        const uint32_t idesc1 = idesc0 | (2u << 29) | (2u << 4);
        const uint64_t desc0 = make_smem_desc(smem_u32(smem), 16, 1024, 2);
        const uint32_t desc_hi = (uint32_t)(desc0 >> 32), lo0 = (uint32_t)desc0;
        const uint32_t sfa = tmem_base + 256, sfb = sfa + 8, hi2 = 2u << 30;
        bool ok = true;
        for (uint32_t b = 0; b < batches && ok; ++b) {
            if (b >= 2) ok = mbar_wait(&bars[b & 1], ((b >> 1) - 1) & 1);       // at most two batches in the queue
#pragma unroll 1
            for (int j = 0; j < kBatch / 4; ++j) {
                const uint32_t a_lo = lo0 + (uint32_t)((j & (kStagesC - 1)) * 2) * (kTileC >> 4), b_lo = a_lo + (kTileC >> 4);
                auto D = [&](uint32_t lo) { return ((uint64_t)desc_hi << 32) | lo; };
                tc_mma_mxf4_pair(tmem_base, D(a_lo), D(b_lo), idesc0, sfa, sfb, 1u);
                tc_mma_mxf4_pair(tmem_base, D(a_lo + 2), D(b_lo + 2), idesc1, sfa | hi2, sfb | hi2, 1u);
                tc_mma_mxf4_pair(tmem_base, D(a_lo + 4), D(b_lo + 4), idesc0, sfa + 4, sfb + 8, 1u);
                tc_mma_mxf4_pair(tmem_base, D(a_lo + 6), D(b_lo + 6), idesc1, (sfa + 4) | hi2, (sfb + 8) | hi2, 1u);
            }
            tc_commit_pair_local(&bars[b & 1]);
        }
        // drain: the last two batches
        for (uint32_t b = batches >= 2 ? batches - 2 : 0; b < batches && ok; ++b) ok = mbar_wait(&bars[b & 1], (b >> 1) & 1);
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();
    if (warp == 0) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, 512);
    }
}

// Diagnostic: one thread waits on a barrier that nothing ever signals.  The bounded wait gives up after its time limit,
// records the status word and the kernel returns normally: the path every kernel of the library takes when a wait
// expires, exercised without a fault.
__global__ void wait_expiry_kernel() {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
        (void)mbar_wait(&bar, 0);            // phase 0 never completes: returns false after the limit, status word set
    }
}

}  // namespace

cudaError_t fetch_fp4_ceiling_status(unsigned int* word) { return device_status_fetch(word); }

}  // namespace mx

extern "C" mxfp4_status mxfp4_selftest_wait_expiry(void* cuda_stream) {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return MXFP4_ERR_CUDA;
    if (major != 10) return MXFP4_ERR_DEVICE;
    mx::wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>();
    return cudaGetLastError() == cudaSuccess ? MXFP4_OK : MXFP4_ERR_CUDA;
}

extern "C" mxfp4_status mxfp4_fp4_ceiling(int64_t mma_per_pair, int64_t* flop_out, void* cuda_stream) {
    // 2e7 instructions per pair are about two seconds of device time: the kernel cannot be pre-empted or stopped early
    if (mma_per_pair <= 0 || mma_per_pair > MXFP4_CEILING_MAX_MMA_PER_PAIR || flop_out == nullptr) return MXFP4_ERR_SHAPE;
    int dev = 0, sms = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return MXFP4_ERR_CUDA;
    if (major != 10) return MXFP4_ERR_DEVICE;
    if (cudaFuncSetAttribute(mx::fp4_ceiling_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mx::kSmemC) != cudaSuccess)
        return MXFP4_ERR_CUDA;
    const int64_t batches = (mma_per_pair + mx::kBatch - 1) / mx::kBatch;
    if (batches > 0x7FFFFFFF) return MXFP4_ERR_SHAPE;
    const int pairs = sms / 2;
    mx::fp4_ceiling_kernel<<<2 * pairs, mx::kThreadsC, mx::kSmemC, static_cast<cudaStream_t>(cuda_stream)>>>((uint32_t)batches);
    if (cudaGetLastError() != cudaSuccess) return MXFP4_ERR_CUDA;
    *flop_out = (int64_t)pairs * batches * mx::kBatch * (2ll * 256 * 256 * 64);
    return MXFP4_OK;
}
