/*
 * mxfp4.h - C ABI of the B200 (sm_100a) MXFP4 linear-layer backward library.
 *
 * The library computes the backward GEMMs of a linear layer y = x W^T,
 *     dX = dY W      (dgrad, reduce over out-features m)
 *     dW = dY^T X    (wgrad, reduce over tokens b)
 * in MXFP4: each operand goes through a blockwise random Hadamard transform
 * along the reduction dimension (one shared sign vector), is quantised to
 * E2M1 values with one E8M0 scale per 32 contiguous elements, and the
 * products run as block-scaled FP4 tensor-core GEMMs ("Training LLMs with
 * MXFP4", Algorithms 1-3).
 *
 * Conventions for every call
 *   - All data pointers are DEVICE pointers owned by the caller.  Nothing the
 *     caller can see is allocated by the library; it never synchronises the
 *     stream (except mxfp4_device_status) and enqueues all work on the CUDA
 *     stream passed as `cuda_stream` (a cudaStream_t cast to void*, NULL = the
 *     legacy default stream).
 *   - Tensors are row-major.  bf16 data, codes and scales must be 16-byte
 *     aligned; leading dimensions must keep every row 16-byte aligned.
 *   - Return value: MXFP4_OK or an error code.  Invalid arguments are reported
 *     as errors, never as undefined behaviour, and every argument check and
 *     tensor-map encoding happens before the first launch: for all codes
 *     except MXFP4_ERR_CUDA nothing was enqueued.  MXFP4_ERR_CUDA may come from
 *     a kernel launch the driver refused after earlier kernels of the same call
 *     were enqueued; outputs are then undefined, but the stream stays ordered
 *     (a call that used its side stream has joined it back).
 *   - Inputs must be finite.  A block containing Inf/NaN gets scale byte 255.
 *   - Same inputs + same seed => bit-identical outputs.
 */
#ifndef MXFP4_B200_H_
#define MXFP4_B200_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define MXFP4_API __attribute__((visibility("default")))
#else
#define MXFP4_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MXFP4_OK = 0,
    MXFP4_ERR_NULL = 1,       /* a required pointer is NULL */
    MXFP4_ERR_SHAPE = 2,      /* a dimension is zero/negative or not divisible as required */
    MXFP4_ERR_ALIGN = 3,      /* a pointer or leading dimension breaks the 16-byte rule */
    MXFP4_ERR_BAD_G = 4,      /* g not in {0, 32, 64, 128, 256} or does not divide the reduce length */
    MXFP4_ERR_MODE = 5,       /* unknown rounding / layout / dtype selector */
    MXFP4_ERR_WORKSPACE = 6,  /* workspace NULL, misaligned or too small */
    MXFP4_ERR_DEVICE = 7,     /* current device is not sm_100 */
    MXFP4_ERR_CUDA = 8,       /* a CUDA runtime / driver call failed */
    MXFP4_ERR_TIMEOUT = 9     /* a bounded device-side wait expired (see mxfp4_device_status) */
} mxfp4_status;

/* rounding: Algorithm 2 (3/4 pre-scale + stochastic rounding; SR with an 8-bit dither and a centred threshold,
 * SR16 with the 16-bit dither of the sm_100a stochastic-rounding convert) or Algorithm 1 (OCP nearest rounding) */
enum { MXFP4_ROUND_SR = 0, MXFP4_ROUND_RN = 1, MXFP4_ROUND_SR16 = 2 };
/* scale layout: LINEAR = [rows, K/32] row-major bytes.
 * NATIVE = the tcgen05 scale-factor tiling consumed by mxfp4_gemm: rows padded to 128, K/32 padded to 4;
 * byte of (row r, block k) at ((r/128)*ceil(K/128) + k/4)*512 + (r%32)*16 + ((r%128)/32)*4 + k%4. */
enum { MXFP4_SF_LINEAR = 0, MXFP4_SF_NATIVE = 1 };
enum { MXFP4_OUT_BF16 = 0, MXFP4_OUT_FP32 = 1 };

/*
 * Blockwise RHT + MXFP4 quantisation of one GEMM operand
 * (Algorithm 3 lines 3-6 followed by Algorithm 2, or Algorithm 1 when rounding = RN).
 *
 *   x          bf16 [rows, cols], leading dimension ld elements (ld >= cols, ld % 8 == 0).
 *   reduce_dim 1: the reduction (K) dimension is `cols` (contiguous).  Output operand is [rows, K = cols].
 *              0: the reduction dimension is `rows`; the output is the TRANSPOSED operand [cols, K = rows]
 *                 (the views of W, dY^T and X^T in Algorithm 3).
 *   g          RHT block size along K: 0 = no transform, else 32/64/128/256; K % max(g, 32) == 0
 *              (K % 128 == 0 for the NATIVE scale layout).  Every contiguous g-chunk v becomes
 *              v diag(S) H_g / sqrt(g), H_g the Sylvester Hadamard matrix (Eq. 4), S derived from `seed`.
 *   rounding   MXFP4_ROUND_SR: per 32 values, shared_exp = floor(log2 amax) - 2, then each value is
 *              multiplied by 3/4, divided by 2^shared_exp and stochastically rounded to E2M1 with an 8-bit
 *              Philox4x32-10 draw r keyed on (seed, stream_tag, element index): up iff 256 frac >= r + 1/2.
 *              MXFP4_ROUND_SR16: the same with a 16-bit dither R, up iff 65536 frac >= 65536 - R (Eq. 2 to
 *              2^-16); the elements 4h..4h+3 of a row share the Philox word whose bytes the SR mode draws for
 *              them, b0..b3: R = 256 b2 + b0, its bit reversal, 256 b3 + b1, its bit reversal.  One convert
 *              instruction rounds four values, which makes this mode the faster one.  MXFP4_ROUND_RN: nearest
 *              rounding (ties to even, saturating at 6) of value / 2^shared_exp, no pre-scale.
 *   seed       drives the sign vector (shared by every operand quantised with the same seed) and SR.
 *   stream_tag separates the SR noise of different operands that share a seed (they must differ between
 *              the two operands of one GEMM for the product to be unbiased, Lemma 3.1).
 *   codes      out, [R, K/2] bytes, two E2M1 codes per byte, even k in the low nibble (R = output rows).
 *   scales     out, E8M0 bytes (value 2^(byte-127)) in `sf_layout`; mxfp4_scale_bytes() gives the size.
 */
MXFP4_API mxfp4_status mxfp4_rht_sr_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim,
                                   int g, int rounding, uint64_t seed, uint32_t stream_tag,
                                   uint8_t* codes, uint8_t* scales, int sf_layout, void* cuda_stream);

/*
 * The transform alone (Algorithm 3 lines 3-6; Section 3.2): writes the fp32 values that the quantiser
 * rounds, y [R, K] row-major, same `reduce_dim`/`g`/`seed` meaning as above.  For inspection and tests.
 */
MXFP4_API mxfp4_status mxfp4_rht(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim,
                       int g, uint64_t seed, float* y, void* cuda_stream);

/*
 * The same quantiser with a transform matrix given by the caller (Section 3.2: the blockwise construction works with
 * any random orthogonal matrix, the RHT is one choice): every contiguous g-chunk v of the reduction dimension becomes
 * v T before quantisation.
 *   T      bf16 [g, g] row-major, DEVICE pointer, 16-byte aligned, g in {32, 64, 128}; applied as given (no 1/sqrt(g)).
 *          The product of two operands is preserved only if both use the same T and T is orthogonal: the caller's duty.
 *   y      NULL, or fp32 [R, K] out (16-byte aligned): then only the transform runs and codes / scales may be NULL.
 *   seed, stream_tag: the SR draws only (there is no sign vector here).  K % 128 == 0 (tensor-core path only),
 *   else MXFP4_ERR_SHAPE.  Everything else as mxfp4_rht_sr_quantize.
 */
MXFP4_API mxfp4_status mxfp4_transform_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim,
                                                int g, const void* T, int rounding, uint64_t seed, uint32_t stream_tag,
                                                uint8_t* codes, uint8_t* scales, int sf_layout, float* y,
                                                void* cuda_stream);

/*
 * Block-scaled FP4 GEMM (MXFP4_GEMM of Algorithm 3 lines 7-8, with the 16/9 of lines 10-11 as alpha):
 *     C[M, N] = alpha * sum_k deq(A)[i, k] * deq(B)[j, k],   deq = E2M1 value * 2^(scale byte - 127)
 *   A_codes [M, K/2], B_codes [N, K/2] packed as above; A_scales / B_scales in the NATIVE layout
 *   (sf_layout must be MXFP4_SF_NATIVE); K % 128 == 0; N % 8 == 0.
 *   C row-major with leading dimension ldc elements, bf16 or fp32 per out_dtype; fp32 accumulation.
 */
MXFP4_API mxfp4_status mxfp4_gemm(const uint8_t* A_codes, const uint8_t* A_scales,
                        const uint8_t* B_codes, const uint8_t* B_scales,
                        int64_t M, int64_t N, int64_t K, int sf_layout, float alpha,
                        void* C, int64_t ldc, int out_dtype, void* cuda_stream);

/* Bytes of device workspace mxfp4_linear_backward needs for these shapes (codes + scales of the four
 * quantised operands). */
MXFP4_API size_t mxfp4_linear_backward_workspace(int64_t b, int64_t m, int64_t n);

/*
 * Algorithm 3: MXFP4 linear-layer backward with the blockwise RHT.
 *   dY bf16 [b, m], X bf16 [b, n], W bf16 [m, n]  ->  dX [b, n], dW [m, n] (bf16 or fp32, dense).
 *   g divides m and b (the two reduction lengths); with g = 0, m % 128 == 0 and b % 128 == 0.
 *   The four operand views are quantised with stream tags 1..4 (dY, W^T, dY^T, X^T) and one shared sign
 *   vector; dX = alpha Q1 Q2^T, dW = alpha Q3 Q4^T with alpha = 16/9 iff rounding = SR or SR16.
 *   workspace: device scratch of at least mxfp4_linear_backward_workspace() bytes, 256-byte aligned;
 *   its contents are overwritten.  Calls sharing a workspace must be stream-ordered.
 *   Ordering: everything the call does is ordered after prior work of `cuda_stream` and before later work of it.
 *   For large shapes the two GEMMs (independent of each other) run side by side: the call forks onto a
 *   library-owned side stream after the quantisers and joins back into `cuda_stream` before it returns (event
 *   record / wait only, no host synchronisation).  The side stream and its two events are created once per host
 *   thread at the first such call; MXFP4_FORK_JOIN=0 in the environment keeps every launch on `cuda_stream`.
 */
MXFP4_API mxfp4_status mxfp4_linear_backward(const void* dY, const void* X, const void* W,
                                   int64_t b, int64_t m, int64_t n, int g, int rounding, uint64_t seed,
                                   void* dX, void* dW, int out_dtype,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Algorithm 3 lines 3-6 alone: the four operand views of one layer (stream tags 1..4: dY, W^T, dY^T, X^T), quantised
 * in ONE launch into `workspace` at the offsets mxfp4_operand_layout reports; lines 7-11 are then two mxfp4_gemm calls
 * (dX = alpha Q1 Q2^T with M = b, N = n, K = m; dW = alpha Q3 Q4^T with M = m, N = n, K = b).  This is what
 * mxfp4_linear_backward does internally; the split form lets a caller time the parts, or keep Q2 (the weights) for
 * several micro-batches that share a seed.  Arguments and errors as mxfp4_linear_backward.
 *   offsets[2 i], offsets[2 i + 1]: byte offsets of the codes and of the scales (NATIVE layout) of view i + 1.
 */
MXFP4_API void mxfp4_operand_layout(int64_t b, int64_t m, int64_t n, size_t offsets[8]);
MXFP4_API mxfp4_status mxfp4_quantize_operands(const void* dY, const void* X, const void* W,
                                               int64_t b, int64_t m, int64_t n, int g, int rounding, uint64_t seed,
                                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Algorithm 3 with the two remaining pieces of a linear layer's backward (problem statement, Section 2:
 * dL/db = 1 dL/dy; micro-batch gradient accumulation):
 *   db:         NULL, or fp32 [m] (16-byte aligned): the bias gradient, column sums of dY in fp32 (not quantised).
 *   accumulate: 0: dW = ..., db = ...;  1: dW += ..., db += ... (out_dtype must be MXFP4_OUT_FP32, else
 *               MXFP4_ERR_MODE).  dX is overwritten in both cases.
 *   workspace:  at least mxfp4_linear_backward_ex_workspace(b, m, n, db != NULL) bytes, 256-byte aligned.
 * Everything else as mxfp4_linear_backward.
 */
MXFP4_API size_t mxfp4_linear_backward_ex_workspace(int64_t b, int64_t m, int64_t n, int with_bias);
MXFP4_API mxfp4_status mxfp4_linear_backward_ex(const void* dY, const void* X, const void* W,
                                      int64_t b, int64_t m, int64_t n, int g, int rounding, uint64_t seed,
                                      void* dX, void* dW, float* db, int out_dtype, int accumulate,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Fused-producer variant (Section 3.2 proposes fusing the transform with the GEMM's operand path): a block-scaled
 * FP4 GEMM whose A operand is transformed and quantised INSIDE the GEMM kernel, never written to global memory:
 *     C[M, N] = alpha * Q(A blockdiag(S H_g / sqrt(g))) deq(B)^T
 *   x, rows, cols, ld, reduce_dim, g, rounding, seed, stream_tag: as in mxfp4_rht_sr_quantize; A = x [M = rows,
 *     K = cols] for reduce_dim 1, A = x^T [M = cols, K = rows] for reduce_dim 0.  g in {32, 64, 128}; K % 256 == 0.
 *   B_codes [N, K/2], B_scales (NATIVE layout): the other operand, quantised beforehand.  N % 8 == 0.
 *   C [M, N], leading dimension ldc, bf16 or fp32.
 * The codes the kernel derives are those mxfp4_rht_sr_quantize would write for the same arguments (the SR draws are
 * keyed on the element index), so the result equals mxfp4_gemm on that call's output.  Every CTA re-quantises the A
 * panel of its 128 x 128 output tile, N / 128 times over the whole product: for wide N this is several times slower
 * than quantising once and is offered for measurement and for narrow N.
 * Errors as mxfp4_rht_sr_quantize and mxfp4_gemm; shapes the kernel does not take give MXFP4_ERR_SHAPE / BAD_G.
 */
MXFP4_API mxfp4_status mxfp4_gemm_fused(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim,
                                        int g, int rounding, uint64_t seed, uint32_t stream_tag,
                                        const uint8_t* B_codes, const uint8_t* B_scales, int64_t N, float alpha,
                                        void* C, int64_t ldc, int out_dtype, void* cuda_stream);

/*
 * Algorithm 3 on the fused-producer kernel: W^T and X^T (lines 4, 6) are quantised by the stand-alone kernel, dY and
 * dY^T (lines 3, 5) inside the two GEMMs.  Arguments, workspace and results as mxfp4_linear_backward, with
 * g in {32, 64, 128}, m % 256 == 0 and b % 256 == 0; codes, and therefore dX and dW, agree with that call's.
 */
MXFP4_API mxfp4_status mxfp4_linear_backward_fused(const void* dY, const void* X, const void* W,
                                                   int64_t b, int64_t m, int64_t n, int g, int rounding, uint64_t seed,
                                                   void* dX, void* dW, int out_dtype,
                                                   void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same backward pass for callers that cannot supply a workspace.  (The paper has no counterpart: this is a
 * property of the library, not of the method.)
 *
 * Who needs it: code that runs where device memory cannot be requested, for instance a hook called while its host
 * framework's memory pool is locked or fully handed out, a plug-in that must not touch the CUDA allocator of the
 * process it lives in, or a tool that has to keep working once device memory is exhausted.  Instead of a caller's
 * buffer the scratch is a fixed array of MXFP4_STATIC_WORKSPACE_BYTES inside the library image; every GPU that loads
 * the library holds that much memory from load to exit, whether or not this call is ever used.
 *
 *   Arguments and results are those of mxfp4_linear_backward without the workspace pair.
 *   Shapes whose mxfp4_linear_backward_workspace(b, m, n) exceeds MXFP4_STATIC_WORKSPACE_BYTES are refused with
 *   MXFP4_ERR_WORKSPACE; nothing is enqueued.
 *   The call allocates nothing, neither on the host nor on the device.
 *   The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that device
 *   current); make that first call outside any stream capture.  That first call is also the moment at which the
 *   CUDA runtime may load the library's kernels and the array itself onto the device (module loading is lazy), which
 *   does need free device memory: a caller that wants the call to survive memory exhaustion makes one warm-up call
 *   per device while memory is still available.  Later calls take nothing from any allocator.
 *   All calls on a device share the one array, which keeps whatever the previous call left in it.  Each call rewrites
 *   every byte it later reads, so nothing needs clearing between calls; but two calls whose kernels can overlap on
 *   the GPU (different streams without ordering) race on it: order them.
 */
#define MXFP4_STATIC_WORKSPACE_BYTES (8u << 20)
MXFP4_API mxfp4_status mxfp4_linear_backward_static(const void* dY, const void* X, const void* W,
                                                    int64_t b, int64_t m, int64_t n, int g, int rounding, uint64_t seed,
                                                    void* dX, void* dW, int out_dtype, void* cuda_stream);

/*
 * FP8 (E4M3) forward pass (Section 4.1, closing remark, and the supplementary section "FP8 Forward Pass Results":
 * the MXFP4 backward pass combined with an E4M3 forward pass).  y = x W^T with both operands quantised to E4M3 under
 * one scale per tensor; the paper names the format, the arithmetic below is this library's reading of it.
 *
 * mxfp4_fp8_quantize: x bf16 [rows, cols] (leading dimension ld; cols and ld multiples of 8).  scale[0] receives
 *   448 / amax(|x|) computed in fp32 (1 for an all-zero tensor), scale[1] the amax itself (it is the call's scratch
 *   word): `scale` points to TWO floats on the device, 8-byte aligned.  codes [rows, cols] bytes receive
 *   E4M3(fp32(x * scale[0])), round-to-nearest-even, saturating at +-448.  Two kernels, no host synchronisation.
 * mxfp4_fp8_gemm: C [M, N] = (sum_k A[i, k] B[j, k]) / (A_scale[0] B_scale[0]); A [M, K], B [N, K] E4M3 bytes, K-major,
 *   K % 128 == 0, N % 8 == 0; the scales are DEVICE pointers (as written by mxfp4_fp8_quantize); fp32 accumulation on the
 *   tensor cores (tcgen05 kind::f8f6f4); C bf16 or fp32, leading dimension ldc.
 * mxfp4_linear_forward_fp8: y [b, m] = x [b, n] W [m, n]^T through the two calls above; n % 128 == 0, m % 8 == 0;
 *   workspace of mxfp4_linear_forward_fp8_workspace(b, n, m) bytes, 256-byte aligned (codes of both operands, scales).
 * Errors as for the other calls (MXFP4_ERR_NULL / _SHAPE / _ALIGN / _MODE / _WORKSPACE / _CUDA).
 */
MXFP4_API mxfp4_status mxfp4_fp8_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, uint8_t* codes, float* scale,
                                          void* cuda_stream);
MXFP4_API mxfp4_status mxfp4_fp8_gemm(const uint8_t* A_codes, const float* A_scale, const uint8_t* B_codes, const float* B_scale,
                                      int64_t M, int64_t N, int64_t K, void* C, int64_t ldc, int out_dtype, void* cuda_stream);
MXFP4_API size_t mxfp4_linear_forward_fp8_workspace(int64_t b, int64_t n, int64_t m);
MXFP4_API mxfp4_status mxfp4_linear_forward_fp8(const void* x, const void* W, int64_t b, int64_t n, int64_t m, void* y, int out_dtype,
                                                void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * MXINT4 elements (Section 3, opening: the analysis "also applies to other low precision datatypes such as MXINT4").
 * An element is a sign-magnitude integer in [-7, 7]; 32 elements along the reduction dimension share one E8M0 scale,
 * chosen by the rule of Algorithms 1 / 2 with emax_elem = 2 (the largest power of two among the elements is 4).
 * MXFP4_ROUND_SR: Algorithm 2 (3/4 pre-scale, stochastic rounding on the integer grid, which is Eq. 1-2 as printed,
 * with the 8-bit draws of the MXFP4 path); MXFP4_ROUND_RN: Algorithm 1 (nearest, ties to even, saturating at 7).
 *
 * mxfp4_int4_quantize: arguments as mxfp4_rht_sr_quantize (same transform, same sign vector, same draws), except:
 *   codes [R, K] is ONE BYTE per element, the integer held as an E4M3 number (the tensor core has no 4-bit integer
 *   type; E4M3 holds -7..7 exactly), scales always in the NATIVE layout, and y_scratch (fp32 [R, K], 16-byte
 *   aligned, caller-owned) receives the transformed values on the way.
 * mxfp4_int4_gemm: C [M, N] = alpha sum_k q_A X_A q_B X_B on the tensor cores (tcgen05 kind::mxf8f6f4, one scale per
 *   32 elements); K % 128 == 0, N % 8 == 0; alpha = 16/9 undoes two 3/4 pre-scales as in Algorithm 3.
 */
MXFP4_API mxfp4_status mxfp4_int4_quantize(const void* x, int64_t rows, int64_t cols, int64_t ld, int reduce_dim, int g, int rounding,
                                           uint64_t seed, uint32_t stream_tag, uint8_t* codes, uint8_t* scales, float* y_scratch,
                                           void* cuda_stream);
MXFP4_API mxfp4_status mxfp4_int4_gemm(const uint8_t* A_codes, const uint8_t* A_scales, const uint8_t* B_codes, const uint8_t* B_scales,
                                       int64_t M, int64_t N, int64_t K, float alpha, void* C, int64_t ldc, int out_dtype,
                                       void* cuda_stream);

/*
 * Measurement aid, not part of the method (the paper has no counterpart): launches a kernel in which every CTA pair
 * issues `mma_per_pair` (rounded up to a multiple of 32) back-to-back 256 x 256 x 64 block-scaled FP4 tensor-core
 * instructions on operands resident in shared memory: no loads, no output.  *flop_out (HOST pointer) receives the
 * floating-point operations the launch performs; time the launch with CUDA events on `cuda_stream` to obtain the
 * on-box ceiling of the FP4 tensor pipe.  mma_per_pair is limited to MXFP4_CEILING_MAX_MMA_PER_PAIR (about two seconds
 * of device time: the kernel cannot be stopped once launched); larger values are refused with MXFP4_ERR_SHAPE.
 * Errors: MXFP4_ERR_SHAPE, MXFP4_ERR_DEVICE, MXFP4_ERR_CUDA.
 */
#define MXFP4_CEILING_MAX_MMA_PER_PAIR 20000000
MXFP4_API mxfp4_status mxfp4_fp4_ceiling(int64_t mma_per_pair, int64_t* flop_out, void* cuda_stream);

/*
 * Diagnostic, not part of the method: launches one warp that waits on a barrier nothing signals.  Every device-side
 * wait of the library is bounded (about two seconds); when one expires the kernel records a status word, unwinds and
 * returns normally.  This call takes exactly that path without any fault: after it, mxfp4_device_status returns
 * MXFP4_ERR_TIMEOUT once (and clears the word), and the context stays usable.  Takes about two seconds of device time.
 */
MXFP4_API mxfp4_status mxfp4_selftest_wait_expiry(void* cuda_stream);

/* Size in bytes of a scale tensor for an operand [rows, K] in the given layout (NATIVE is padded). */
MXFP4_API size_t mxfp4_scale_bytes(int64_t rows, int64_t K, int sf_layout);

/* Synchronises `cuda_stream`, then reads and clears the device status word that kernels set when a
 * bounded wait expires.  Returns MXFP4_OK, MXFP4_ERR_TIMEOUT or MXFP4_ERR_CUDA.  The only call that blocks. */
MXFP4_API mxfp4_status mxfp4_device_status(void* cuda_stream);

MXFP4_API const char* mxfp4_status_string(mxfp4_status status);

#ifdef __cplusplus
}
#endif
#endif /* MXFP4_B200_H_ */
