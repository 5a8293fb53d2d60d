// C-ABI entry points (include/mxfp4.h): argument validation, tensor-map set-up and kernel launches.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdio>
#include <cstdlib>
#include <mutex>

#include "../../include/mxfp4.h"
#include "kernels.h"
#include "ptx.cuh"

namespace {

using mx::GemmArgs;
using mx::QuantArgs;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct Runtime {
    std::once_flag once;
    mxfp4_status status = MXFP4_OK;
    EncodeTiledFn encode = nullptr;
    bool gemm_pair = true;       // CTA-pair GEMM (gemm_pair.cu); MXFP4_GEMM_PAIR=0 selects the 1-CTA kernel (gemm.cu)
    std::mutex mu;
    static constexpr int kMaxDevices = 64;
    mxfp4_status dev_status[kMaxDevices];
    bool dev_done[kMaxDevices] = {};
};
Runtime g_rt;

// Set-up: once per process the driver entry point for tensor-map encoding and the environment switches; once per
// device (kernel attributes belong to the device's context) the capability check and the shared-memory opt-in.
mxfp4_status runtime_init() {
    std::call_once(g_rt.once, [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || fn == nullptr ||
            qres != cudaDriverEntryPointSuccess) {
            g_rt.status = MXFP4_ERR_CUDA;
            return;
        }
        g_rt.encode = reinterpret_cast<EncodeTiledFn>(fn);
        const char* pair = getenv("MXFP4_GEMM_PAIR");
        g_rt.gemm_pair = !(pair != nullptr && pair[0] == '0');
    });
    if (g_rt.status != MXFP4_OK) return g_rt.status;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= Runtime::kMaxDevices) return MXFP4_ERR_CUDA;
    // Tensor-map encoding is a driver call and needs the device's context current on the CALLING thread.  A thread
    // that has only inherited the device number (a framework's worker thread) may not have it bound yet: selecting the
    // device it already names binds the primary context.  Done once per thread and device.
    static thread_local int bound_dev = -1;
    if (bound_dev != dev) {
        if (cudaSetDevice(dev) != cudaSuccess) return MXFP4_ERR_CUDA;
        bound_dev = dev;
    }
    std::lock_guard<std::mutex> lock(g_rt.mu);
    if (!g_rt.dev_done[dev]) {
        int major = 0;
        mxfp4_status st = MXFP4_OK;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) st = MXFP4_ERR_CUDA;
        else if (major != 10) st = MXFP4_ERR_DEVICE;
        else if (mx::gemm_init() != cudaSuccess || mx::gemm_pair_init() != cudaSuccess || mx::quant_tc_init() != cudaSuccess ||
                 mx::gemm_fused_init() != cudaSuccess || mx::gemm_f8_init() != cudaSuccess)
            st = MXFP4_ERR_CUDA;
        g_rt.dev_status[dev] = st;
        g_rt.dev_done[dev] = true;
    }
    return g_rt.dev_status[dev];
}

// Side stream and events for running the two independent GEMMs of a backward call side by side (fork / join around
// the caller's stream): the second GEMM's CTAs move onto SMs as the first one's last wave drains.  One set per host
// thread, created at its first large call and kept; on any failure the call simply stays on the caller's stream.
struct ForkJoin {
    bool tried = false, ok = false;
    int device = -1;
    cudaStream_t side = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
};
ForkJoin* fork_join() {
    static thread_local ForkJoin fj;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    if (!fj.tried) {
        fj.tried = true;
        fj.device = dev;
        int lo = 0, hi = 0;
        fj.ok = cudaDeviceGetStreamPriorityRange(&lo, &hi) == cudaSuccess &&
                cudaStreamCreateWithPriority(&fj.side, cudaStreamNonBlocking, lo) == cudaSuccess &&
                cudaEventCreateWithFlags(&fj.fork, cudaEventDisableTiming) == cudaSuccess &&
                cudaEventCreateWithFlags(&fj.join, cudaEventDisableTiming) == cudaSuccess;
        const char* e = getenv("MXFP4_FORK_JOIN");
        if (e != nullptr && e[0] == '0') fj.ok = false;
    }
    return fj.ok && fj.device == dev ? &fj : nullptr;
}

// With MXFP4_DEBUG set in the environment a failing CUDA call is named on stderr (the ABI only returns MXFP4_ERR_CUDA).
mxfp4_status cuda_status(cudaError_t e, const char* where) {
    if (e == cudaSuccess) return MXFP4_OK;
    if (getenv("MXFP4_DEBUG") != nullptr) fprintf(stderr, "mxfp4: %s failed: %s\n", where, cudaGetErrorString(e));
    return MXFP4_ERR_CUDA;
}

mxfp4_status encode_status(CUresult r, const char* where) {
    if (r == CUDA_SUCCESS) return MXFP4_OK;
    if (getenv("MXFP4_DEBUG") != nullptr) fprintf(stderr, "mxfp4: tensor-map encoding failed (%s): CUresult %d\n", where, (int)r);
    return MXFP4_ERR_CUDA;
}

// MXFP4_OVERLAP: 0 (default) = serial form (quantise everything, then the two GEMMs); 1 = overlapped form with the
// cheaper head first; 2 / 3 = overlapped with dX / dW first.  Read at every call so that one process can compare the
// forms.  The overlapped form is off by default because it measured no faster (the GEMM runs at the board's power
// limit, so quantiser work done beside it slows it by about the time that was hidden).
// MXFP4_FORCE_LITE=1: every pair GEMM and every grouped quantiser launch uses the small build of its kernel (tests use
// this to put the small builds through the ragged and tiny shapes that the overlapped form itself never sees).
bool force_lite() {
    const char* e = getenv("MXFP4_FORCE_LITE");
    return e != nullptr && e[0] == '1';
}

// MXFP4_DUAL_DY: 1 (default) = one read of dL/dy for its two views where that pays (large layers, or a bias gradient
// wanted); 0 = always separate tile lists (two reads); 2 = always one read.
int dual_setting() {
    const char* e = getenv("MXFP4_DUAL_DY");
    if (e == nullptr || e[0] == '\0') return 1;
    return e[0] >= '0' && e[0] <= '2' ? e[0] - '0' : 1;
}

int overlap_setting() {
    const char* e = getenv("MXFP4_OVERLAP");
    if (e == nullptr || e[0] == '\0') return 0;
    return e[0] >= '0' && e[0] <= '3' ? e[0] - '0' : 0;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool valid_g(int g) { return g == 0 || g == 32 || g == 64 || g == 128 || g == 256; }
int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

size_t scale_bytes(int64_t rows, int64_t K, int layout) {
    if (rows <= 0 || K <= 0) return 0;
    if (layout == MXFP4_SF_NATIVE) return (size_t)(((rows + 127) / 128) * ((K + 127) / 128) * 512);
    return (size_t)(rows * ((K + 31) / 32));
}

mxfp4_status check_quant(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim, int g) {
    if (x == nullptr) return MXFP4_ERR_NULL;
    if (rows <= 0 || cols <= 0 || ld < cols) return MXFP4_ERR_SHAPE;
    if (reduce_dim != 0 && reduce_dim != 1) return MXFP4_ERR_MODE;
    if (!valid_g(g)) return MXFP4_ERR_BAD_G;
    const int64_t K = reduce_dim == 1 ? cols : rows;
    if (K % 32 != 0) return MXFP4_ERR_SHAPE;
    if (g != 0 && K % g != 0) return MXFP4_ERR_BAD_G;
    if (!aligned16(x) || ld % 8 != 0 || cols % 8 != 0) return MXFP4_ERR_ALIGN;
    if (rows * cols / 32 > (int64_t)0x7FFFFFFF * 256) return MXFP4_ERR_SHAPE;
    return MXFP4_OK;
}

// Tensor map over a byte matrix [rows, row_bytes]: box = 128 bytes of a row x box_rows rows, 128-byte swizzle.
mxfp4_status make_bytes_map(CUtensorMap* map, const uint8_t* codes, int64_t rows, int64_t row_bytes, int box_rows);
// ... over packed E2M1 codes [rows, K/2] bytes.
mxfp4_status make_codes_map(CUtensorMap* map, const uint8_t* codes, int64_t rows, int64_t K, int box_rows) {
    return make_bytes_map(map, codes, rows, K / 2, box_rows);
}
mxfp4_status make_bytes_map(CUtensorMap* map, const uint8_t* codes, int64_t rows, int64_t row_bytes, int box_rows) {
    const int64_t K = 2 * row_bytes;
    const cuuint64_t dims[2] = {(cuuint64_t)row_bytes, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)mx::kGemmBKBytes, (cuuint32_t)box_rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    const CUresult r = g_rt.encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(codes), dims, strides, box, elem_strides,
                                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS && getenv("MXFP4_DEBUG") != nullptr)
        fprintf(stderr, "mxfp4: codes map: ptr %p rows %lld K %lld box_rows %d\n", (const void*)codes, (long long)rows, (long long)K, box_rows);
    return encode_status(r, "codes");
}

// Tensor map over the bf16 input [rows, cols] (leading dimension ld): box = 64 columns x 128 rows, 128-byte swizzle.
// Only built when the tensor-core quantiser can take the call; otherwise the CUDA-core kernels read x directly.
void attach_input_map(QuantArgs& a) {
    a.has_tmap = false;
    const int64_t K = a.reduce_dim == 1 ? a.cols : a.rows;
    if (!(a.g == 32 || a.g == 64 || a.g == 128 || a.g == 256) || K % 128 != 0) return;
    if (a.rows > 0x7FFFFFFF || a.cols > 0x7FFFFFFF) return;
    const cuuint64_t dims[2] = {(cuuint64_t)a.cols, (cuuint64_t)a.rows};
    const cuuint64_t strides[1] = {(cuuint64_t)a.ld * 2};
    const cuuint32_t box[2] = {64, 128};
    const cuuint32_t elem_strides[2] = {1, 1};
    const CUresult r = g_rt.encode(&a.tmap_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(a.x), dims, strides, box,
                                   elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    a.has_tmap = r == CUDA_SUCCESS;
}

// Tensor map over the output C [M, N] for the pair kernel's stores: box = 64 bytes of a row x 32 rows, 64-byte swizzle.
bool make_output_map(CUtensorMap* map, void* C, int64_t M, int64_t N, int64_t ldc, bool fp32) {
    const int64_t es = fp32 ? 4 : 2;
    if ((reinterpret_cast<uintptr_t>(C) & 15u) != 0 || (ldc * es) % 16 != 0 || M > 0x7FFFFFFF || N > 0x7FFFFFFF) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)(ldc * es)};
    const cuuint32_t box[2] = {(cuuint32_t)(64 / es), 32};
    const cuuint32_t elem_strides[2] = {1, 1};
    const CUresult r = g_rt.encode(map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, C, dims, strides,
                                   box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B,
                                   CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Everything a GEMM launch needs (tensor maps included), built without touching the device.
mxfp4_status gemm_prepare(GemmArgs& a, const uint8_t* A_codes, const uint8_t* A_scales, const uint8_t* B_codes, const uint8_t* B_scales,
                          int64_t M, int64_t N, int64_t K, float alpha, void* C, int64_t ldc, int out_dtype, int accumulate) {
    mxfp4_status st = make_codes_map(&a.tmap_a, A_codes, M, K, mx::kGemmBM);
    if (st != MXFP4_OK) return st;
    st = make_codes_map(&a.tmap_b, B_codes, N, K, mx::kGemmBN);
    if (st != MXFP4_OK) return st;
    a.sfa = A_scales; a.sfb = B_scales;
    a.M = M; a.N = N; a.K = K;
    a.alpha = alpha; a.C = C; a.ldc = ldc; a.out_fp32 = out_dtype == MXFP4_OUT_FP32;
    a.accumulate = accumulate;
    a.use_pair = g_rt.gemm_pair && M > 128;                   // one 128-row tile gives a pair nothing to share
    a.has_tmap_c = false;
    a.lite = a.use_pair && force_lite();
    if (a.use_pair) {
        st = make_codes_map(&a.tmap_b_half, B_codes, N, K, 128);
        if (st != MXFP4_OK) return st;
        a.has_tmap_c = make_output_map(&a.tmap_c, C, M, N, ldc, a.out_fp32 != 0);
    }
    return MXFP4_OK;
}

mxfp4_status gemm_launch(const GemmArgs& a, cudaStream_t stream) {
    return cuda_status(a.use_pair ? mx::launch_gemm_pair(a, stream) : mx::launch_gemm(a, stream), a.use_pair ? "pair GEMM launch" : "GEMM launch");
}

mxfp4_status gemm_impl(const uint8_t* A_codes, const uint8_t* A_scales, const uint8_t* B_codes, const uint8_t* B_scales, int64_t M,
                       int64_t N, int64_t K, float alpha, void* C, int64_t ldc, int out_dtype, cudaStream_t stream,
                       int accumulate = 0) {
    GemmArgs a;
    const mxfp4_status st = gemm_prepare(a, A_codes, A_scales, B_codes, B_scales, M, N, K, alpha, C, ldc, out_dtype, accumulate);
    return st != MXFP4_OK ? st : gemm_launch(a, stream);
}

// C = alpha Q(RHT(A)) deq(B)^T with A = x (reduce_dim 1) or x^T (reduce_dim 0) quantised inside the GEMM kernel.
mxfp4_status gemm_fused_impl(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim, int g, int rounding, uint64_t seed,
                             uint32_t stream_tag, const uint8_t* B_codes, const uint8_t* B_scales, int64_t N, float alpha, void* C,
                             int64_t ldc, int out_dtype, cudaStream_t stream) {
    QuantArgs q{x, rows, cols, ld, reduce_dim, g, rounding, seed, stream_tag, nullptr, nullptr, 1, nullptr};
    attach_input_map(q);
    mx::FusedGemmArgs a;
    a.tmap_x = q.tmap_x; a.has_tmap_x = q.has_tmap;
    a.M = reduce_dim == 1 ? rows : cols; a.K = reduce_dim == 1 ? cols : rows; a.N = N;
    a.sfb = B_scales; a.alpha = alpha; a.C = C; a.ldc = ldc; a.out_fp32 = out_dtype == MXFP4_OUT_FP32;
    a.g = g; a.reduce_dim = reduce_dim; a.rounding = rounding; a.seed = seed; a.stream_tag = stream_tag;
    if (!mx::gemm_fused_eligible(a)) return MXFP4_ERR_SHAPE;
    const mxfp4_status st = make_codes_map(&a.tmap_b, B_codes, N, a.K, 128);
    if (st != MXFP4_OK) return st;
    return mx::launch_gemm_fused(a, stream) == cudaSuccess ? MXFP4_OK : MXFP4_ERR_CUDA;
}

struct Workspace {
    size_t codes[4], scales[4], total;
};
// Operand views of Algorithm 3: Q1 = dY [b, K=m], Q2 = W^T [n, K=m], Q3 = dY^T [m, K=b], Q4 = X^T [n, K=b].
Workspace plan_workspace(int64_t b, int64_t m, int64_t n) {
    const int64_t R[4] = {b, n, m, n}, K[4] = {m, m, b, b};
    Workspace w;
    size_t off = 0;
    for (int i = 0; i < 4; ++i) {
        w.codes[i] = off;
        off += (size_t)round_up(R[i] * K[i] / 2, 1024);
        w.scales[i] = off;
        off += (size_t)round_up((int64_t)scale_bytes(R[i], K[i], MXFP4_SF_NATIVE), 1024);
    }
    w.total = off;
    return w;
}

}  // namespace

extern "C" {

const char* mxfp4_status_string(mxfp4_status s) {
    switch (s) {
        case MXFP4_OK: return "ok";
        case MXFP4_ERR_NULL: return "null pointer";
        case MXFP4_ERR_SHAPE: return "bad shape";
        case MXFP4_ERR_ALIGN: return "bad alignment";
        case MXFP4_ERR_BAD_G: return "bad RHT block size g";
        case MXFP4_ERR_MODE: return "bad mode selector";
        case MXFP4_ERR_WORKSPACE: return "bad workspace";
        case MXFP4_ERR_DEVICE: return "device is not sm_100";
        case MXFP4_ERR_CUDA: return "CUDA call failed";
        case MXFP4_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

size_t mxfp4_scale_bytes(int64_t rows, int64_t K, int sf_layout) { return scale_bytes(rows, K, sf_layout); }

mxfp4_status mxfp4_rht_sr_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim, int g, int rounding,
                                   uint64_t seed, uint32_t stream_tag, uint8_t* codes, uint8_t* scales, int sf_layout,
                                   void* cuda_stream) {
    if (codes == nullptr || scales == nullptr) return MXFP4_ERR_NULL;
    mxfp4_status st = check_quant(x, rows, cols, ld, reduce_dim, g);
    if (st != MXFP4_OK) return st;
    if (rounding != MXFP4_ROUND_SR && rounding != MXFP4_ROUND_RN && rounding != MXFP4_ROUND_SR16) return MXFP4_ERR_MODE;
    if (sf_layout != MXFP4_SF_LINEAR && sf_layout != MXFP4_SF_NATIVE) return MXFP4_ERR_MODE;
    if (!aligned16(codes)) return MXFP4_ERR_ALIGN;
    if ((st = runtime_init()) != MXFP4_OK) return st;
    QuantArgs a{x, rows, cols, ld, reduce_dim, g, rounding, seed, stream_tag, codes, scales, sf_layout == MXFP4_SF_NATIVE, nullptr};
    attach_input_map(a);
    return mx::launch_quantize(a, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? MXFP4_OK : MXFP4_ERR_CUDA;
}

mxfp4_status mxfp4_rht(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim, int g, uint64_t seed, float* y,
                       void* cuda_stream) {
    if (y == nullptr) return MXFP4_ERR_NULL;
    mxfp4_status st = check_quant(x, rows, cols, ld, reduce_dim, g);
    if (st != MXFP4_OK) return st;
    if (!aligned16(y)) return MXFP4_ERR_ALIGN;
    if ((st = runtime_init()) != MXFP4_OK) return st;
    QuantArgs a{x, rows, cols, ld, reduce_dim, g, 0, seed, 0u, nullptr, nullptr, 0, y};
    attach_input_map(a);
    return mx::launch_rht_dump(a, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? MXFP4_OK : MXFP4_ERR_CUDA;
}

mxfp4_status mxfp4_transform_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim, int g, const void* T,
                                      int rounding, uint64_t seed, uint32_t stream_tag, uint8_t* codes, uint8_t* scales,
                                      int sf_layout, float* y, void* cuda_stream) {
    if (T == nullptr || ((codes == nullptr || scales == nullptr) && y == nullptr)) return MXFP4_ERR_NULL;
    mxfp4_status st = check_quant(x, rows, cols, ld, reduce_dim, g);
    if (st != MXFP4_OK) return st;
    if (g != 32 && g != 64 && g != 128) return MXFP4_ERR_BAD_G;
    if (rounding != MXFP4_ROUND_SR && rounding != MXFP4_ROUND_RN && rounding != MXFP4_ROUND_SR16) return MXFP4_ERR_MODE;
    if (sf_layout != MXFP4_SF_LINEAR && sf_layout != MXFP4_SF_NATIVE) return MXFP4_ERR_MODE;
    if (!aligned16(T) || (codes && !aligned16(codes)) || (y && !aligned16(y))) return MXFP4_ERR_ALIGN;
    if ((st = runtime_init()) != MXFP4_OK) return st;
    QuantArgs a{x, rows, cols, ld, reduce_dim, g, rounding, seed, stream_tag, codes, scales, sf_layout == MXFP4_SF_NATIVE, y};
    a.custom_t = T;
    attach_input_map(a);
    if (!mx::quant_tc_eligible(a)) return MXFP4_ERR_SHAPE;            // the given-matrix transform runs on the tensor-core path only
    return mx::launch_quantize_tc(a, y != nullptr, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? MXFP4_OK : MXFP4_ERR_CUDA;
}

mxfp4_status mxfp4_gemm(const uint8_t* A_codes, const uint8_t* A_scales, const uint8_t* B_codes, const uint8_t* B_scales, int64_t M,
                        int64_t N, int64_t K, int sf_layout, float alpha, void* C, int64_t ldc, int out_dtype, void* cuda_stream) {
    if (!A_codes || !A_scales || !B_codes || !B_scales || !C) return MXFP4_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || K % 128 != 0 || N % 8 != 0 || ldc < N) return MXFP4_ERR_SHAPE;
    if (M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > 0x7FFFFFFF) return MXFP4_ERR_SHAPE;
    if (sf_layout != MXFP4_SF_NATIVE) return MXFP4_ERR_MODE;
    if (out_dtype != MXFP4_OUT_BF16 && out_dtype != MXFP4_OUT_FP32) return MXFP4_ERR_MODE;
    if (!aligned16(A_codes) || !aligned16(B_codes) || !aligned16(A_scales) || !aligned16(B_scales) || !aligned16(C)) return MXFP4_ERR_ALIGN;
    if (ldc % (out_dtype == MXFP4_OUT_FP32 ? 4 : 8) != 0) return MXFP4_ERR_ALIGN;
    const mxfp4_status st = runtime_init();
    if (st != MXFP4_OK) return st;
    return gemm_impl(A_codes, A_scales, B_codes, B_scales, M, N, K, alpha, C, ldc, out_dtype, static_cast<cudaStream_t>(cuda_stream));
}

mxfp4_status mxfp4_gemm_fused(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim, int g, int rounding, uint64_t seed,
                              uint32_t stream_tag, const uint8_t* B_codes, const uint8_t* B_scales, int64_t N, float alpha, void* C,
                              int64_t ldc, int out_dtype, void* cuda_stream) {
    if (!B_codes || !B_scales || !C) return MXFP4_ERR_NULL;
    mxfp4_status st = check_quant(x, rows, cols, ld, reduce_dim, g);
    if (st != MXFP4_OK) return st;
    if (g != 32 && g != 64 && g != 128) return MXFP4_ERR_BAD_G;
    if (rounding != MXFP4_ROUND_SR && rounding != MXFP4_ROUND_RN && rounding != MXFP4_ROUND_SR16) return MXFP4_ERR_MODE;
    if (out_dtype != MXFP4_OUT_BF16 && out_dtype != MXFP4_OUT_FP32) return MXFP4_ERR_MODE;
    const int64_t K = reduce_dim == 1 ? cols : rows;
    if (N <= 0 || N % 8 != 0 || ldc < N || K % 256 != 0 || N > 0x7FFFFFFF || rows > 0x7FFFFFFF || cols > 0x7FFFFFFF) return MXFP4_ERR_SHAPE;
    if (!aligned16(B_codes) || !aligned16(B_scales) || !aligned16(C) || ldc % (out_dtype == MXFP4_OUT_FP32 ? 4 : 8) != 0) return MXFP4_ERR_ALIGN;
    if ((st = runtime_init()) != MXFP4_OK) return st;
    return gemm_fused_impl(x, rows, cols, ld, reduce_dim, g, rounding, seed, stream_tag, B_codes, B_scales, N, alpha, C, ldc, out_dtype,
                           static_cast<cudaStream_t>(cuda_stream));
}

size_t mxfp4_linear_backward_workspace(int64_t b, int64_t m, int64_t n) {
    if (b <= 0 || m <= 0 || n <= 0) return 0;
    return plan_workspace(b, m, n).total;
}

}  // extern "C"

namespace {
// Algorithm 3 lines 3-6: the four operand views, stream tags 1..4, one sign vector (same seed) for all of them.
struct Overlap {
    int first;            // in: product to run first (0 = dX, 1 = dW), its operands are quantised up front; out: -1 if the call fell back to the serial form
    ForkJoin* fj;
    bool forked = false;  // the side stream holds work that the caller's stream has to wait for
};
mxfp4_status quantize_operands_impl(const void* dY, const void* X, const void* W, int64_t b, int64_t m, int64_t n, int g, int rounding,
                                    uint64_t seed, uint8_t* const c[4], uint8_t* const s[4], cudaStream_t stream, Overlap* ov = nullptr,
                                    float* col_sums = nullptr, bool* col_sums_done = nullptr) {
    QuantArgs q[4] = {
        {dY, b, m, m, 1, g, rounding, seed, 1u, c[0], s[0], 1, nullptr},   // dY   [b, K = m]
        {W, m, n, n, 0, g, rounding, seed, 2u, c[1], s[1], 1, nullptr},    // W^T  [n, K = m]
        {dY, b, m, m, 0, g, rounding, seed, 3u, c[2], s[2], 1, nullptr},   // dY^T [m, K = b]
        {X, b, n, n, 0, g, rounding, seed, 4u, c[3], s[3], 1, nullptr},    // X^T  [n, K = b]
    };
    bool all_tc = true;
    for (int i = 0; i < 4; ++i) {
        attach_input_map(q[i]);
        all_tc = all_tc && mx::quant_tc_eligible(q[i]);
    }
    if (ov != nullptr && ov->first >= 0 && all_tc && g != 256) {
        // Overlapped form: the operands of the product that runs first are quantised by the full-size kernel on the
        // caller's stream; the other product's operands by the small build on the side stream, which shares the SMs
        // with the small build of the first GEMM (launched by the caller of this function).
        const int a0 = ov->first == 0 ? 0 : 2, b0 = 2 - a0;             // views (a0, a0 + 1) first, (b0, b0 + 1) hidden
        const QuantArgs head[2] = {q[a0], q[a0 + 1]}, tail[2] = {q[b0], q[b0 + 1]};
        if (cuda_status(mx::launch_quantize_tc_group(head, 2, false, stream), "quantiser launch (first product)") != MXFP4_OK) return MXFP4_ERR_CUDA;
        if (cudaEventRecord(ov->fj->fork, stream) != cudaSuccess || cudaStreamWaitEvent(ov->fj->side, ov->fj->fork, 0) != cudaSuccess) {
            ov->first = -1;                          // could not fork: the rest of the call stays on the caller's stream
            return cuda_status(mx::launch_quantize_tc_group(tail, 2, false, stream), "quantiser launch (second product)");
        }
        ov->forked = true;
        return cuda_status(mx::launch_quantize_tc_group(tail, 2, false, ov->fj->side, true), "small quantiser launch (second product)");
    }
    if (ov != nullptr) ov->first = -1;
    // (worth a second launch only when dL/dy is large: below 2^25 elements, or when the column sums are not wanted from
    // it either, the four views go as one tile list in one launch, which is what the small layers' short kernels prefer)
    const int dual_mode = dual_setting();
    if (all_tc && g != 256 && !force_lite() && (dual_mode == 2 || (dual_mode == 1 && (b * m >= (int64_t(1) << 25) || col_sums != nullptr)))) {
        // dL/dy feeds lines 3 and 5: its two views come from ONE read of it; W^T and X^T in a second launch
        const QuantArgs dy[2] = {q[0], q[2]}, wx[2] = {q[1], q[3]};
        if (cuda_status(mx::launch_quantize_tc_group(dy, 2, false, stream, false, true, col_sums), "quantiser launch (both views of dY)") != MXFP4_OK) return MXFP4_ERR_CUDA;
        if (col_sums != nullptr && col_sums_done != nullptr) *col_sums_done = true;     // the bias gradient's first pass rode along
        return cuda_status(mx::launch_quantize_tc_group(wx, 2, false, stream), "quantiser launch (W, X)");
    }
    if (all_tc)                                     // the four views of the call in one launch
        return cuda_status(mx::launch_quantize_tc_group(q, 4, false, stream, g != 256 && force_lite()), "grouped quantiser launch");
    for (int i = 0; i < 4; ++i)
        if (cuda_status(mx::launch_quantize(q[i], stream), "quantiser launch") != MXFP4_OK) return MXFP4_ERR_CUDA;
    return MXFP4_OK;
}

// Argument checks shared by the entry points that take a whole layer.
mxfp4_status check_layer(const void* dY, const void* X, const void* W, int64_t b, int64_t m, int64_t n, int g, int rounding) {
    if (!dY || !X || !W) return MXFP4_ERR_NULL;
    if (b <= 0 || m <= 0 || n <= 0) return MXFP4_ERR_SHAPE;
    if (!valid_g(g)) return MXFP4_ERR_BAD_G;
    if (m % 128 != 0 || b % 128 != 0 || n % 8 != 0) return MXFP4_ERR_SHAPE;       // both reduce lengths feed the GEMM (K % 128)
    if (g != 0 && (m % g != 0 || b % g != 0)) return MXFP4_ERR_BAD_G;
    if (rounding != MXFP4_ROUND_SR && rounding != MXFP4_ROUND_RN && rounding != MXFP4_ROUND_SR16) return MXFP4_ERR_MODE;
    if (!aligned16(dY) || !aligned16(X) || !aligned16(W)) return MXFP4_ERR_ALIGN;
    return MXFP4_OK;
}

// Algorithm 3, optionally with the bias gradient (db != NULL) and accumulation into dW and db.
mxfp4_status linear_backward_impl(const void* dY, const void* X, const void* W, int64_t b, int64_t m, int64_t n, int g, int rounding,
                                  uint64_t seed, void* dX, void* dW, float* db, int out_dtype, int accumulate, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream) {
    if (!dY || !X || !W || !dX || !dW) return MXFP4_ERR_NULL;
    if (b <= 0 || m <= 0 || n <= 0) return MXFP4_ERR_SHAPE;
    if (!valid_g(g)) return MXFP4_ERR_BAD_G;
    if (m % 128 != 0 || b % 128 != 0 || n % 8 != 0) return MXFP4_ERR_SHAPE;       // both reduce lengths feed the GEMM (K % 128)
    if (g != 0 && (m % g != 0 || b % g != 0)) return MXFP4_ERR_BAD_G;
    if (rounding != MXFP4_ROUND_SR && rounding != MXFP4_ROUND_RN && rounding != MXFP4_ROUND_SR16) return MXFP4_ERR_MODE;
    if (out_dtype != MXFP4_OUT_BF16 && out_dtype != MXFP4_OUT_FP32) return MXFP4_ERR_MODE;
    if (accumulate != 0 && accumulate != 1) return MXFP4_ERR_MODE;
    if (accumulate == 1 && out_dtype != MXFP4_OUT_FP32) return MXFP4_ERR_MODE;      // accumulation is defined on fp32 gradients
    if (!aligned16(dY) || !aligned16(X) || !aligned16(W) || !aligned16(dX) || !aligned16(dW) || (db && !aligned16(db))) return MXFP4_ERR_ALIGN;
    Workspace ws = plan_workspace(b, m, n);
    const size_t bias_off = ws.total;
    if (db != nullptr) ws.total += (size_t)round_up((int64_t)mx::bias_grad_workspace(b, m), 1024);
    if (workspace == nullptr || workspace_bytes < ws.total || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MXFP4_ERR_WORKSPACE;
    mxfp4_status st = runtime_init();
    if (st != MXFP4_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    uint8_t *c[4], *s[4];
    for (int i = 0; i < 4; ++i) { c[i] = base + ws.codes[i]; s[i] = base + ws.scales[i]; }
    // lines 7-11: two MXFP4 GEMMs; the 16/9 un-does the two 3/4 pre-scales of Algorithm 2.
    const float alpha = rounding != MXFP4_ROUND_RN ? 16.0f / 9.0f : 1.0f;       // both SR modes carry the 3/4 pre-scale
    // Every tensor map is encoded before the first launch, so an encoding failure leaves nothing enqueued.
    GemmArgs gx, gw;
    if ((st = gemm_prepare(gx, c[0], s[0], c[1], s[1], b, n, m, alpha, dX, n, out_dtype, 0)) != MXFP4_OK) return st;   // dX is never accumulated
    if ((st = gemm_prepare(gw, c[2], s[2], c[3], s[3], m, n, b, alpha, dW, n, out_dtype, accumulate)) != MXFP4_OK) return st;
    const int64_t waves_dx = ((b + 255) / 256) * ((n + 255) / 256), waves_dw = ((m + 255) / 256) * ((n + 255) / 256);
    // Large problems (never the ones the fixed-scratch variant accepts) use a side stream.
    ForkJoin* fj = ws.total > (size_t)MXFP4_STATIC_WORKSPACE_BYTES && waves_dx >= 74 && waves_dw >= 74 ? fork_join() : nullptr;
    // Overlapped form (Section 3.2: the transform need not cost GEMM time): quantise the operands of one product, then
    // run that product's GEMM while the other product's operands are quantised on the same SMs (small builds of both
    // kernels share an SM: the GEMM keeps the FP4 pipe, the quantiser takes the idle issue slots and ALUs), then the
    // second GEMM.  The product whose operands are the smaller half goes first, so that more of the quantiser work hides.
    const int overlap_mode = overlap_setting();
    Overlap ov{-1, fj};
    if (fj != nullptr && overlap_mode != 0 && gx.use_pair && gw.use_pair && g != 0 && g != 256) {
        const int64_t head_dx = b * m + n * m, head_dw = m * b + n * b;       // elements quantised before the first GEMM can start
        ov.first = overlap_mode == 2 ? 0 : overlap_mode == 3 ? 1 : (head_dx <= head_dw ? 0 : 1);
    }
    float* bias_partial = db != nullptr ? reinterpret_cast<float*>(base + bias_off) : nullptr;
    bool bias_fused = false;
    if ((st = quantize_operands_impl(dY, X, W, b, m, n, g, rounding, seed, c, s, stream, &ov, bias_partial, &bias_fused)) != MXFP4_OK) {
        if (ov.forked && (cudaEventRecord(fj->join, fj->side) != cudaSuccess || cudaStreamWaitEvent(stream, fj->join, 0) != cudaSuccess)) return MXFP4_ERR_CUDA;
        return st;
    }
    if (ov.first >= 0) {
        GemmArgs& g1 = ov.first == 0 ? gx : gw;
        GemmArgs& g2 = ov.first == 0 ? gw : gx;
        g1.lite = true;                              // shares its SMs with the small quantiser running on the side stream
        st = gemm_launch(g1, stream);
        const bool joined = cudaEventRecord(fj->join, fj->side) == cudaSuccess && cudaStreamWaitEvent(stream, fj->join, 0) == cudaSuccess;
        if (!joined) return MXFP4_ERR_CUDA;
        if (st == MXFP4_OK) st = gemm_launch(g2, stream);
        fj = nullptr;                                // joined already
    } else {
        if (fj != nullptr && (cudaEventRecord(fj->fork, stream) != cudaSuccess || cudaStreamWaitEvent(fj->side, fj->fork, 0) != cudaSuccess))
            fj = nullptr;                            // the side stream was not given anything yet: stay on the caller's stream
        st = gemm_launch(gx, stream);
        if (st == MXFP4_OK) st = gemm_launch(gw, fj != nullptr ? fj->side : stream);
    }
    // dL/db = 1 dL/dy (problem statement): column sums of dY, after the GEMMs on the caller's stream
    // (when the dual-view quantiser launch has already summed every 128-row band of dY, only the bands remain to be added)
    if (st == MXFP4_OK && db != nullptr)
        st = bias_fused ? cuda_status(mx::launch_bias_finish(bias_partial, m, (int)(b / 128), accumulate, db, stream), "bias gradient launch")
                        : cuda_status(mx::launch_bias_grad(dY, b, m, m, accumulate, db, bias_partial, stream), "bias gradient launch");
    // The join is made whatever happened after the fork, so that the side stream never runs unordered with the caller's.
    if (fj != nullptr && (cudaEventRecord(fj->join, fj->side) != cudaSuccess || cudaStreamWaitEvent(stream, fj->join, 0) != cudaSuccess))
        return MXFP4_ERR_CUDA;
    return st;
}
}  // namespace

extern "C" {

mxfp4_status mxfp4_linear_backward(const void* dY, const void* X, const void* W, int64_t b, int64_t m, int64_t n, int g, int rounding,
                                   uint64_t seed, void* dX, void* dW, int out_dtype, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream) {
    return linear_backward_impl(dY, X, W, b, m, n, g, rounding, seed, dX, dW, nullptr, out_dtype, 0, workspace, workspace_bytes, cuda_stream);
}

size_t mxfp4_linear_backward_ex_workspace(int64_t b, int64_t m, int64_t n, int with_bias) {
    if (b <= 0 || m <= 0 || n <= 0) return 0;
    return plan_workspace(b, m, n).total + (with_bias ? (size_t)round_up((int64_t)mx::bias_grad_workspace(b, m), 1024) : 0);
}

mxfp4_status mxfp4_linear_backward_ex(const void* dY, const void* X, const void* W, int64_t b, int64_t m, int64_t n, int g, int rounding,
                                      uint64_t seed, void* dX, void* dW, float* db, int out_dtype, int accumulate, void* workspace,
                                      size_t workspace_bytes, void* cuda_stream) {
    return linear_backward_impl(dY, X, W, b, m, n, g, rounding, seed, dX, dW, db, out_dtype, accumulate, workspace, workspace_bytes, cuda_stream);
}

mxfp4_status mxfp4_linear_backward_fused(const void* dY, const void* X, const void* W, int64_t b, int64_t m, int64_t n, int g, int rounding,
                                         uint64_t seed, void* dX, void* dW, int out_dtype, void* workspace, size_t workspace_bytes,
                                         void* cuda_stream) {
    if (!dY || !X || !W || !dX || !dW) return MXFP4_ERR_NULL;
    if (b <= 0 || m <= 0 || n <= 0) return MXFP4_ERR_SHAPE;
    if (g != 32 && g != 64 && g != 128) return MXFP4_ERR_BAD_G;
    if (m % 256 != 0 || b % 256 != 0 || n % 8 != 0) return MXFP4_ERR_SHAPE;          // the fused kernel steps K by 256
    if (rounding != MXFP4_ROUND_SR && rounding != MXFP4_ROUND_RN && rounding != MXFP4_ROUND_SR16) return MXFP4_ERR_MODE;
    if (out_dtype != MXFP4_OUT_BF16 && out_dtype != MXFP4_OUT_FP32) return MXFP4_ERR_MODE;
    if (!aligned16(dY) || !aligned16(X) || !aligned16(W) || !aligned16(dX) || !aligned16(dW)) return MXFP4_ERR_ALIGN;
    const Workspace ws = plan_workspace(b, m, n);
    if (workspace == nullptr || workspace_bytes < ws.total || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MXFP4_ERR_WORKSPACE;
    mxfp4_status st = runtime_init();
    if (st != MXFP4_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    // lines 4 and 6: the B operands (W^T, X^T) are quantised once by the stand-alone kernel
    QuantArgs q[2] = {
        {W, m, n, n, 0, g, rounding, seed, 2u, base + ws.codes[1], base + ws.scales[1], 1, nullptr},
        {X, b, n, n, 0, g, rounding, seed, 4u, base + ws.codes[3], base + ws.scales[3], 1, nullptr},
    };
    for (int i = 0; i < 2; ++i) {
        attach_input_map(q[i]);
        if (!mx::quant_tc_eligible(q[i])) return MXFP4_ERR_SHAPE;
    }
    if (mx::launch_quantize_tc_group(q, 2, false, stream) != cudaSuccess) return MXFP4_ERR_CUDA;
    const float alpha = rounding != MXFP4_ROUND_RN ? 16.0f / 9.0f : 1.0f;
    // lines 3 + 7 and 5 + 8: dY is transformed and rounded inside the GEMMs (stream tags 1 and 3)
    st = gemm_fused_impl(dY, b, m, m, 1, g, rounding, seed, 1u, q[0].codes, q[0].scales, n, alpha, dX, n, out_dtype, stream);
    if (st != MXFP4_OK) return st;
    return gemm_fused_impl(dY, b, m, m, 0, g, rounding, seed, 3u, q[1].codes, q[1].scales, n, alpha, dW, n, out_dtype, stream);
}

void mxfp4_operand_layout(int64_t b, int64_t m, int64_t n, size_t offsets[8]) {
    if (offsets == nullptr) return;
    for (int i = 0; i < 8; ++i) offsets[i] = 0;
    if (b <= 0 || m <= 0 || n <= 0) return;
    const Workspace ws = plan_workspace(b, m, n);
    for (int i = 0; i < 4; ++i) { offsets[2 * i] = ws.codes[i]; offsets[2 * i + 1] = ws.scales[i]; }
}

mxfp4_status mxfp4_quantize_operands(const void* dY, const void* X, const void* W, int64_t b, int64_t m, int64_t n, int g, int rounding,
                                     uint64_t seed, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    mxfp4_status st = check_layer(dY, X, W, b, m, n, g, rounding);
    if (st != MXFP4_OK) return st;
    const Workspace ws = plan_workspace(b, m, n);
    if (workspace == nullptr || workspace_bytes < ws.total || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MXFP4_ERR_WORKSPACE;
    if ((st = runtime_init()) != MXFP4_OK) return st;
    uint8_t* base = static_cast<uint8_t*>(workspace);
    uint8_t *c[4], *s[4];
    for (int i = 0; i < 4; ++i) { c[i] = base + ws.codes[i]; s[i] = base + ws.scales[i]; }
    return quantize_operands_impl(dY, X, W, b, m, n, g, rounding, seed, c, s, static_cast<cudaStream_t>(cuda_stream));
}

// ------------------------------------------------------------------------------------------ FP8 (E4M3) forward pass
mxfp4_status mxfp4_fp8_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, float* scale, void* cuda_stream) {
    if (!x || !codes || !scale) return MXFP4_ERR_NULL;
    if (rows <= 0 || cols <= 0 || ld < cols || cols % 8 != 0 || ld % 8 != 0) return MXFP4_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(codes) || (reinterpret_cast<uintptr_t>(scale) & 7u) != 0) return MXFP4_ERR_ALIGN;
    const mxfp4_status st = runtime_init();
    if (st != MXFP4_OK) return st;
    return cuda_status(mx::launch_fp8_quantize(x, rows, cols, ld, codes, scale, static_cast<cudaStream_t>(cuda_stream)), "FP8 quantiser launch");
}

namespace {
mxfp4_status gemm8_impl(const uint8_t* A, const uint8_t* B, const uint8_t* sfa, const uint8_t* sfb, const float* sa, const float* sb,
                        int64_t M, int64_t N, int64_t K, float alpha, void* C, int64_t ldc, int out_dtype, cudaStream_t stream) {
    mx::Gemm8Args a;
    mxfp4_status st = make_bytes_map(&a.tmap_a, A, M, K, 128);
    if (st != MXFP4_OK) return st;
    if ((st = make_bytes_map(&a.tmap_b, B, N, K, 256)) != MXFP4_OK) return st;
    a.block_scaled = sfa != nullptr;
    a.sfa = sfa; a.sfb = sfb; a.scale_a = sa; a.scale_b = sb;
    a.M = M; a.N = N; a.K = K; a.alpha = alpha; a.C = C; a.ldc = ldc; a.out_fp32 = out_dtype == MXFP4_OUT_FP32;
    return cuda_status(mx::launch_gemm_f8(a, stream), "8-bit GEMM launch");
}
mxfp4_status check_gemm8(const void* A, const void* B, const void* C, int64_t M, int64_t N, int64_t K, int64_t ldc, int out_dtype) {
    if (!A || !B || !C) return MXFP4_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || K % 128 != 0 || N % 8 != 0 || ldc < N) return MXFP4_ERR_SHAPE;
    if (M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > 0x7FFFFFFF) return MXFP4_ERR_SHAPE;
    if (out_dtype != MXFP4_OUT_BF16 && out_dtype != MXFP4_OUT_FP32) return MXFP4_ERR_MODE;
    if (!aligned16(A) || !aligned16(B) || !aligned16(C) || ldc % (out_dtype == MXFP4_OUT_FP32 ? 4 : 8) != 0) return MXFP4_ERR_ALIGN;
    return MXFP4_OK;
}
}  // namespace

mxfp4_status mxfp4_fp8_gemm(const uint8_t* A_codes, const float* A_scale, const uint8_t* B_codes, const float* B_scale, int64_t M, int64_t N,
                            int64_t K, void* C, int64_t ldc, int out_dtype, void* cuda_stream) {
    if (!A_scale || !B_scale) return MXFP4_ERR_NULL;
    mxfp4_status st = check_gemm8(A_codes, B_codes, C, M, N, K, ldc, out_dtype);
    if (st != MXFP4_OK) return st;
    if ((st = runtime_init()) != MXFP4_OK) return st;
    return gemm8_impl(A_codes, B_codes, nullptr, nullptr, A_scale, B_scale, M, N, K, 1.0f, C, ldc, out_dtype, static_cast<cudaStream_t>(cuda_stream));
}

size_t mxfp4_linear_forward_fp8_workspace(int64_t b, int64_t n, int64_t m) {
    if (b <= 0 || n <= 0 || m <= 0) return 0;
    return (size_t)(round_up(b * n, 1024) + round_up(m * n, 1024) + 1024);      // codes of x, codes of W, the two scale pairs
}

mxfp4_status mxfp4_linear_forward_fp8(const void* x, const void* W, int64_t b, int64_t n, int64_t m, void* y, int out_dtype,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!x || !W) return MXFP4_ERR_NULL;
    mxfp4_status st = check_gemm8(x, W, y, b, m, n, m, out_dtype);                 // y [b, m] = x [b, K = n] W [m, K = n]^T
    if (st != MXFP4_OK) return st;
    if (workspace == nullptr || workspace_bytes < mxfp4_linear_forward_fp8_workspace(b, n, m) || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
        return MXFP4_ERR_WORKSPACE;
    if ((st = runtime_init()) != MXFP4_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* base = static_cast<uint8_t*>(workspace);
    uint8_t* cx = base;
    uint8_t* cw = cx + round_up(b * n, 1024);
    float* sc = reinterpret_cast<float*>(cw + round_up(m * n, 1024));              // [0..1] x: scale, amax; [2..3] W
    if ((st = cuda_status(mx::launch_fp8_quantize(x, b, n, n, cx, sc, stream), "FP8 quantiser launch (x)")) != MXFP4_OK) return st;
    if ((st = cuda_status(mx::launch_fp8_quantize(W, m, n, n, cw, sc + 2, stream), "FP8 quantiser launch (W)")) != MXFP4_OK) return st;
    return gemm8_impl(cx, cw, nullptr, nullptr, sc, sc + 2, b, m, n, 1.0f, y, m, out_dtype, stream);
}

// ------------------------------------------------------------------------------------------ MXINT4 elements
mxfp4_status mxfp4_int4_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim, int g, int rounding, uint64_t seed,
                                 uint32_t stream_tag, uint8_t* codes, uint8_t* scales, float* y_scratch, void* cuda_stream) {
    if (!codes || !scales || !y_scratch) return MXFP4_ERR_NULL;
    mxfp4_status st = check_quant(x, rows, cols, ld, reduce_dim, g);
    if (st != MXFP4_OK) return st;
    if (rounding != MXFP4_ROUND_SR && rounding != MXFP4_ROUND_RN) return MXFP4_ERR_MODE;
    if (!aligned16(codes) || !aligned16(y_scratch)) return MXFP4_ERR_ALIGN;
    if ((st = runtime_init()) != MXFP4_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the transform is the MXFP4 path's own (its fp32 output, rounded once); only the element format differs
    QuantArgs a{x, rows, cols, ld, reduce_dim, g, 0, seed, 0u, nullptr, nullptr, 0, y_scratch};
    attach_input_map(a);
    if ((st = cuda_status(mx::launch_rht_dump(a, stream), "transform launch")) != MXFP4_OK) return st;
    const int64_t R = reduce_dim == 1 ? rows : cols, K = reduce_dim == 1 ? cols : rows;
    return cuda_status(mx::launch_mxint4_quantize(y_scratch, R, K, rounding, seed, stream_tag, codes, scales, stream), "MXINT4 quantiser launch");
}

mxfp4_status mxfp4_int4_gemm(const uint8_t* A_codes, const uint8_t* A_scales, const uint8_t* B_codes, const uint8_t* B_scales, int64_t M,
                             int64_t N, int64_t K, float alpha, void* C, int64_t ldc, int out_dtype, void* cuda_stream) {
    if (!A_scales || !B_scales) return MXFP4_ERR_NULL;
    mxfp4_status st = check_gemm8(A_codes, B_codes, C, M, N, K, ldc, out_dtype);
    if (st != MXFP4_OK) return st;
    if (!aligned16(A_scales) || !aligned16(B_scales)) return MXFP4_ERR_ALIGN;
    if ((st = runtime_init()) != MXFP4_OK) return st;
    return gemm8_impl(A_codes, B_codes, A_scales, B_scales, nullptr, nullptr, M, N, K, alpha, C, ldc, out_dtype, static_cast<cudaStream_t>(cuda_stream));
}

mxfp4_status mxfp4_device_status(void* cuda_stream) {
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return MXFP4_ERR_CUDA;
    unsigned int word = 0;
    cudaError_t (*const fetch[])(unsigned int*) = {mx::fetch_gemm_status, mx::fetch_gemm_pair_status, mx::fetch_quant_tc_status,
                                                   mx::fetch_fp4_ceiling_status, mx::fetch_gemm_fused_status, mx::fetch_gemm_f8_status};
    for (auto f : fetch) {
        unsigned int w = 0;
        if (f(&w) != cudaSuccess) return MXFP4_ERR_CUDA;
        word |= w;
    }
    if (word != 0) return MXFP4_ERR_TIMEOUT;
    return MXFP4_OK;
}

}  // extern "C"
