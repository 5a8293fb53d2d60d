/*
 * CPU oracle for the MXFP4 linear-layer backward pass ("Training LLMs with MXFP4").
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the
 * method that the CUDA library is checked against.  It shares no code, table
 * or header with the CUDA path and must never be called from it.  Only the
 * test-suite, the smoke check and the CPU-baseline leg of the benchmark may
 * load it.
 *
 * Everything is written in the order and notation of the paper:
 *   Eq. 4 / Section 3.2   Sylvester Hadamard matrix, x <- x diag(S) H_g / sqrt(g)
 *   Algorithm 1           OCP nearest-rounding MX quantizer  (rounding = RN)
 *   Algorithm 2           3/4 pre-scale + stochastic rounding (rounding = SR)
 *   Eq. 1-2, Appendix     SR as the two-point law between grid neighbours
 *   Algorithm 3           the four transformed operand views, two GEMMs, x16/9
 *
 * Arithmetic is fp64.  There is no blocking, fusion or reordering: the
 * Hadamard transform is an explicit g x g matrix product, the E2M1 grid is an
 * enumerated table, SR compares a uniform integer draw with the fractional
 * distance to the lower grid neighbour, and the GEMM is a triple loop over
 * dequantised operands.  OpenMP pragmas only parallelise independent rows.
 *
 * Readings of points the paper leaves open (each is restated where used):
 *   - H_g is the +-1 Sylvester matrix of order g (a power of two) times
 *     1/sqrt(g); the transform is block diagonal over contiguous g-chunks of
 *     the reduction dimension, identical for both GEMM operands.
 *   - The transformed value is rounded once to fp32 ("pre-quantisation value").
 *   - shared_exp = floor(log2 amax) - 2, clamped to [-127, 127]; an all-zero
 *     block takes -127.  The scale byte is OCP E8M0: byte = shared_exp + 127.
 *   - SR acts on the exact real w = (3/4) V_i / X; with f <= |w| < c the grid
 *     neighbours and frac = (|w| - f)/(c - f), round up iff
 *     frac >= (r + 1/2)/256,  r a uniform 8-bit integer from Philox4x32-10
 *     keyed on (seed, element index).  This is Eq. 2 with the dither
 *     delta = 1/2 - (r + 1/2)/256 in (-1/2, 1/2): ceil iff x + delta >= floor(x) + 1/2.
 *   - A second SR reading (rounding = 2, "SR16"): the same two-point law with a
 *     16-bit dither R per element, round up iff frac >= (65536 - R)/65536, so
 *     P(up) = floor(65536 frac)/65536.  The four elements 4h..4h+3 share one
 *     Philox word with bytes b0..b3 (low to high): element 4h takes
 *     R = 256 b2 + b0, element 4h+1 the same 16 bits in reversed order,
 *     element 4h+2 takes R = 256 b3 + b1, element 4h+3 that one reversed (the
 *     top eight bits of the four dithers are four different bytes).
 *     PROVENANCE: the two-point law and P(up) are the paper's; the LAYOUT of
 *     the draw (which bytes form R, the bit reversal for odd elements) is not a
 *     reading of the paper.  It is the behaviour of the sm_100a
 *     stochastic-rounding convert instruction, observed on the GPU, and is
 *     restated here only so that the optional SR16 mode can be compared code
 *     by code.  Agreement with orc_sr16_* therefore shows that the CUDA path
 *     uses that instruction as described, not that the description follows
 *     from the paper; what the paper fixes for SR16 (unbiasedness, the
 *     two-point law, independent noise) is checked on the GPU's output without
 *     these functions.  The contract reading is SR (8-bit, Eq. 2) above.
 *   - RN is round-to-nearest, ties to the code with even mantissa bit,
 *     saturating at 6.
 *   - The sign bit of the input is kept (a negative value may round to -0).
 *
 * Pins (tests/, "not gpu"): H H^T = g I; GEMM invariance under the shared RHT;
 * hand-worked RN and SR cases; OCP scale examples; exact enumeration of
 * E[SR(w)]; Var = (c-a)(a-f); Philox known answers; the Hadamard tail bound by
 * brute force; clip fraction of Algorithm 1; E[GEMM] = (9/16) A B^T.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_API __attribute__((visibility("default")))

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): counter-based generator */
/* ------------------------------------------------------------------------- */

ORC_API void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Counter layout used by the method: key = (seed lo, seed hi);
 * counter = (index lo, index hi, stream_tag, domain).
 * domain 0: sign vector (stream_tag 0).  domain 1: SR draws. */
static void philox_call(uint64_t seed, uint64_t index, uint32_t stream_tag, uint32_t domain, uint32_t out[4])
{
    uint32_t ctr[4] = { (uint32_t)index, (uint32_t)(index >> 32), stream_tag, domain };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    orc_philox4x32_10(ctr, key, out);
}

/* Algorithm 3, line 2: one sign vector S in {+1,-1}^g per backward call.
 * Bit j of the 128-bit Philox output of call j/128 (word (j/32)%4, bit j%32);
 * S_j = 1 - 2 bit_j. */
ORC_API void orc_sign_vector(uint64_t seed, int g, int8_t *S)
{
    for (int j = 0; j < g; ++j) {
        uint32_t out[4];
        philox_call(seed, (uint64_t)(j >> 7), 0u, 0u, out);
        uint32_t bit = (out[(j >> 5) & 3] >> (j & 31)) & 1u;
        S[j] = (int8_t)(1 - 2 * (int)bit);
    }
}

/* The 8-bit SR draw of element `i` (linear index in the K-major output view):
 * Philox call i/16, byte i%16 counted low to high through words 0..3. */
ORC_API uint32_t orc_sr_draw(uint64_t seed, uint32_t stream_tag, uint64_t i)
{
    uint32_t out[4];
    philox_call(seed, i >> 4, stream_tag, 1u, out);
    uint32_t f = (uint32_t)(i & 15u);
    return (out[f >> 2] >> (8u * (f & 3u))) & 0xFFu;
}

static uint32_t reverse16(uint32_t v)
{
    uint32_t o = 0;
    for (int i = 0; i < 16; ++i) o |= ((v >> i) & 1u) << (15 - i);
    return o;
}

/* The 16-bit dither of element `i` in the SR16 reading: Philox call i/16, word (i%16)/4 with bytes b0..b3;
 * elements 4h, 4h+2 take 256 b2 + b0 and 256 b3 + b1, elements 4h+1, 4h+3 the bit reversal of their left neighbour's.
 * This byte pairing and the reversal are the hardware convert's, observed on the GPU; the paper does not fix them. */
ORC_API uint32_t orc_sr16_draw(uint64_t seed, uint32_t stream_tag, uint64_t i)
{
    uint32_t out[4];
    philox_call(seed, i >> 4, stream_tag, 1u, out);
    uint32_t word = out[(i >> 2) & 3u];
    uint32_t b0 = word & 0xFFu, b1 = (word >> 8) & 0xFFu, b2 = (word >> 16) & 0xFFu, b3 = word >> 24;
    uint32_t j = (uint32_t)(i & 3u);
    uint32_t R = (j < 2u) ? (256u * b2 + b0) : (256u * b3 + b1);
    return (j & 1u) ? reverse16(R) : R;
}

/* ------------------------------------------------------------------------- */
/* Eq. 4: Sylvester Hadamard matrix, un-normalised (+-1 entries)              */
/* ------------------------------------------------------------------------- */

/* H_1 = [1]; H_{2n} = [[H_n, H_n], [H_n, -H_n]], built by the recursion itself. */
ORC_API int orc_hadamard(int g, int8_t *H /* g*g, row-major */)
{
    if (g < 1 || (g & (g - 1)) != 0) return -1;
    H[0] = 1;
    for (int n = 1; n < g; n *= 2) {
        /* grow the n x n block in the top-left corner to 2n x 2n (row stride g) */
        for (int i = 0; i < n; ++i)
            for (int j = 0; j < n; ++j) {
                int8_t h = H[i * g + j];
                H[i * g + (j + n)] = h;
                H[(i + n) * g + j] = h;
                H[(i + n) * g + (j + n)] = (int8_t)-h;
            }
    }
    return 0;
}

static double bf16_to_double(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Section 3.2 / Algorithm 3 lines 3-6 for one operand viewed as [R, K] with K
 * the reduction dimension: every contiguous g-chunk v of a row becomes
 *     y_j = (1/sqrt(g)) sum_i v_i S_i H[i][j],
 * an explicit matrix product in fp64, rounded once to fp32.  g = 0 means no
 * transform (y = v).  x is bf16 (raw 16-bit patterns) with element (r, k) at
 * x[r*stride_r + k*stride_k], so the transposed views of Algorithm 3 are read
 * in place. */
ORC_API int orc_rht(const uint16_t *x, int64_t R, int64_t K, int64_t stride_r, int64_t stride_k,
                    int g, uint64_t seed, float *y /* [R, K] row-major */)
{
    if (g == 0) {
#pragma omp parallel for schedule(static)
        for (int64_t r = 0; r < R; ++r)
            for (int64_t k = 0; k < K; ++k)
                y[r * K + k] = (float)bf16_to_double(x[r * stride_r + k * stride_k]);
        return 0;
    }
    if (g < 2 || (g & (g - 1)) != 0 || K % g != 0) return -1;
    int8_t *H = (int8_t *)malloc((size_t)g * g);
    int8_t *S = (int8_t *)malloc((size_t)g);
    if (!H || !S) { free(H); free(S); return -2; }
    orc_hadamard(g, H);
    orc_sign_vector(seed, g, S);
    const double inv_sqrt_g = 1.0 / sqrt((double)g);
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r) {
        double v[256];
        for (int64_t k0 = 0; k0 < K; k0 += g) {
            for (int i = 0; i < g; ++i)
                v[i] = bf16_to_double(x[r * stride_r + (k0 + i) * stride_k]) * (double)S[i];
            for (int j = 0; j < g; ++j) {
                double s = 0.0;
                for (int i = 0; i < g; ++i)
                    s += v[i] * (double)H[i * g + j];
                y[r * K + k0 + j] = (float)(s * inv_sqrt_g);
            }
        }
    }
    free(H); free(S);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* E2M1 element format and E8M0 scale (Section 2.1, Table 1, Section 2.5)     */
/* ------------------------------------------------------------------------- */

/* 1 sign, 2 exponent (bias 1), 1 mantissa bit.  Magnitudes by code 0..7. */
/* Section 3.2, last paragraph: the blockwise construction works with ANY orthogonal g x g matrix in place of
 * diag(S) H_g / sqrt(g).  Every contiguous g-chunk v of a row becomes y_j = sum_i v_i T[i][j], T given as bf16
 * (raw 16-bit patterns, row-major g x g): explicit product in fp64, rounded once to fp32. */
ORC_API int orc_transform(const uint16_t *x, int64_t R, int64_t K, int64_t stride_r, int64_t stride_k,
                          int g, const uint16_t *T, float *y /* [R, K] row-major */)
{
    if (g < 1 || K % g != 0) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r)
        for (int64_t c = 0; c < K / g; ++c)
            for (int j = 0; j < g; ++j) {
                double acc = 0.0;
                for (int i = 0; i < g; ++i)
                    acc += bf16_to_double(x[r * stride_r + (c * g + i) * stride_k]) * bf16_to_double(T[i * g + j]);
                y[r * K + c * g + j] = (float)acc;
            }
    return 0;
}

static const double E2M1_GRID[8] = { 0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0 };

ORC_API double orc_e2m1_value(uint32_t code)
{
    double v = E2M1_GRID[code & 7u];
    return (code & 8u) ? -v : v;
}

/* Algorithm 1/2 lines 1-2 for MXFP4 (emax_elem = 2):
 * shared_exp = floor(log2 amax) - 2, clamped to [-127, 127]; amax = 0 takes
 * the lower clamp; returns the E8M0 byte shared_exp + 127 (255 = not finite). */
ORC_API uint32_t orc_e8m0_from_amax(float amax)
{
    if (!(amax == amax) || isinf(amax)) return 255u;
    if (amax == 0.0f) return 0u;
    int ex;
    (void)frexp((double)amax, &ex);      /* amax = m 2^ex, m in [0.5, 1)  =>  floor(log2 amax) = ex - 1 */
    int shared_exp = (ex - 1) - 2;
    if (shared_exp < -127) shared_exp = -127;
    if (shared_exp > 127) shared_exp = 127;
    return (uint32_t)(shared_exp + 127);
}

/* stochastic_round_to_FP4 (Algorithm 2 line 5) on the exact real w, |w| <= 6:
 * f <= |w| < c neighbours on the enumerated grid; Eq. 2 in units of the local
 * grid step with delta = 1/2 - (r + 1/2)/256: up iff frac + delta >= 1/2. */
ORC_API uint32_t orc_sr_round(double w, uint32_t r)
{
    uint32_t sign = signbit(w) ? 8u : 0u;
    double a = fabs(w);
    if (a >= 6.0) return sign | 7u;                       /* unreachable after the 3/4 pre-scale */
    uint32_t lo = 0;
    while (lo + 1 < 8 && E2M1_GRID[lo + 1] <= a) ++lo;    /* f = grid[lo] <= a < grid[lo+1] = c */
    double f = E2M1_GRID[lo], c = E2M1_GRID[lo + 1];
    double frac = (a - f) / (c - f);
    int up = frac * 256.0 >= ((double)r + 0.5);
    return sign | (lo + (uint32_t)up);
}

/* The same two-point law with a 16-bit dither R (SR16 reading): up iff frac >= (65536 - R)/65536;
 * over uniform R the probability of rounding up is floor(65536 frac)/65536.  |w| >= 6 saturates. */
ORC_API uint32_t orc_sr16_round(double w, uint32_t R)
{
    uint32_t sign = signbit(w) ? 8u : 0u;
    double a = fabs(w);
    if (a >= 6.0) return sign | 7u;
    uint32_t lo = 0;
    while (lo + 1 < 8 && E2M1_GRID[lo + 1] <= a) ++lo;
    double f = E2M1_GRID[lo], c = E2M1_GRID[lo + 1];
    double frac = (a - f) / (c - f);
    int up = frac * 65536.0 >= 65536.0 - (double)R;
    return sign | (lo + (uint32_t)up);
}

/* quantize_to_LP (Algorithm 1 line 4): nearest, ties to even mantissa bit,
 * saturating at the largest normal 6. */
ORC_API uint32_t orc_rn_round(double w)
{
    uint32_t sign = signbit(w) ? 8u : 0u;
    double a = fabs(w);
    if (a >= 6.0) return sign | 7u;
    uint32_t lo = 0;
    while (lo + 1 < 8 && E2M1_GRID[lo + 1] <= a) ++lo;
    double f = E2M1_GRID[lo], c = E2M1_GRID[lo + 1];
    double mid = 0.5 * (f + c);
    uint32_t code;
    if (a < mid) code = lo;
    else if (a > mid) code = lo + 1;
    else code = (lo & 1u) ? lo + 1 : lo;                  /* tie: even code has mantissa bit 0 */
    return sign | code;
}

/* Algorithm 1 (rounding = 1, RN) or Algorithm 2 (rounding = 0, SR; rounding = 2, SR16) applied to
 * every 32 consecutive entries of each row of y [R, K] (fp32 pre-quantisation
 * values).  codes: one 4-bit code per byte [R, K]; scales: E8M0 [R, K/32]. */
ORC_API int orc_quantize_rows(const float *y, int64_t R, int64_t K, int rounding,
                              uint64_t seed, uint32_t stream_tag, const int64_t *row_ids,
                              uint8_t *codes, uint8_t *scales);

ORC_API int orc_quantize(const float *y, int64_t R, int64_t K, int rounding,
                         uint64_t seed, uint32_t stream_tag,
                         uint8_t *codes, uint8_t *scales)
{
    return orc_quantize_rows(y, R, K, rounding, seed, stream_tag, NULL, codes, scales);
}

/* Same, for a subset of the rows of a larger operand: row_ids[r] is the row index in the full K-major
 * operand (it only enters through the element index that keys the SR draw); NULL = 0..R-1. */
ORC_API int orc_quantize_rows(const float *y, int64_t R, int64_t K, int rounding,
                              uint64_t seed, uint32_t stream_tag, const int64_t *row_ids,
                              uint8_t *codes, uint8_t *scales)
{
    if (K % 32 != 0) return -1;
    const int64_t nblk = K / 32;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r) {
        for (int64_t b = 0; b < nblk; ++b) {
            const float *V = y + r * K + b * 32;
            float amax = 0.0f;
            int finite = 1;
            for (int i = 0; i < 32; ++i) {
                float av = fabsf(V[i]);
                if (!(av == av) || isinf(av)) finite = 0;
                if (av > amax) amax = av;
            }
            uint32_t byte = finite ? orc_e8m0_from_amax(amax) : 255u;
            scales[r * nblk + b] = (uint8_t)byte;
            if (byte == 255u) { memset(codes + r * K + b * 32, 0, 32); continue; }
            int shared_exp = (int)byte - 127;
            for (int i = 0; i < 32; ++i) {
                int64_t idx = r * K + b * 32 + i;
                int64_t elem = (row_ids ? row_ids[r] : r) * K + b * 32 + i;   /* index in the full operand */
                if (rounding == 0) {
                    double w = ldexp(0.75 * (double)V[i], -shared_exp);   /* (3/4) V_i / X, exact */
                    codes[idx] = (uint8_t)orc_sr_round(w, orc_sr_draw(seed, stream_tag, (uint64_t)elem));
                } else if (rounding == 2) {
                    double w = ldexp(0.75 * (double)V[i], -shared_exp);
                    codes[idx] = (uint8_t)orc_sr16_round(w, orc_sr16_draw(seed, stream_tag, (uint64_t)elem));
                } else {
                    double w = ldexp((double)V[i], -shared_exp);          /* V_i / X, exact */
                    codes[idx] = (uint8_t)orc_rn_round(w);
                }
            }
        }
    }
    return 0;
}

/* Two codes per byte, element with even k in the low nibble. */
ORC_API void orc_pack(const uint8_t *codes, int64_t n, uint8_t *packed)
{
    for (int64_t i = 0; i < n / 2; ++i)
        packed[i] = (uint8_t)((codes[2 * i] & 0xF) | ((codes[2 * i + 1] & 0xF) << 4));
}

/* value(code) * 2^(byte - 127) */
ORC_API void orc_dequantize(const uint8_t *codes, const uint8_t *scales, int64_t R, int64_t K, double *out)
{
    const int64_t nblk = K / 32;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r)
        for (int64_t k = 0; k < K; ++k)
            out[r * K + k] = ldexp(orc_e2m1_value(codes[r * K + k]), (int)scales[r * nblk + k / 32] - 127);
}

/* ------------------------------------------------------------------------- */
/* MXFP4_GEMM: C[i][j] = alpha sum_k deq(A)[i][k] deq(B)[j][k], fp64           */
/* ------------------------------------------------------------------------- */

/* rows/cols select the output entries to compute (NULL = all); each output
 * depends on one row of A and one row of B, so sampling is exact. */
ORC_API void orc_gemm(const uint8_t *A_codes, const uint8_t *A_scales,
                      const uint8_t *B_codes, const uint8_t *B_scales,
                      int64_t M, int64_t N, int64_t K, double alpha,
                      const int64_t *rows, int64_t n_rows, const int64_t *cols, int64_t n_cols,
                      double *C /* [n_rows, n_cols] */)
{
    const int64_t nblk = K / 32;
    if (!rows) n_rows = M;
    if (!cols) n_cols = N;
    double *Bd = (double *)malloc((size_t)n_cols * K * sizeof(double));
#pragma omp parallel for schedule(static)
    for (int64_t jj = 0; jj < n_cols; ++jj) {
        int64_t j = cols ? cols[jj] : jj;
        for (int64_t k = 0; k < K; ++k)
            Bd[jj * K + k] = ldexp(orc_e2m1_value(B_codes[j * K + k]), (int)B_scales[j * nblk + k / 32] - 127);
    }
#pragma omp parallel
    {
        double *Ad = (double *)malloc((size_t)K * sizeof(double));
#pragma omp for schedule(static)
        for (int64_t ii = 0; ii < n_rows; ++ii) {
            int64_t i = rows ? rows[ii] : ii;
            for (int64_t k = 0; k < K; ++k)
                Ad[k] = ldexp(orc_e2m1_value(A_codes[i * K + k]), (int)A_scales[i * nblk + k / 32] - 127);
            for (int64_t jj = 0; jj < n_cols; ++jj) {
                double s = 0.0;
                for (int64_t k = 0; k < K; ++k)
                    s += Ad[k] * Bd[jj * K + k];
                C[ii * n_cols + jj] = alpha * s;
            }
        }
        free(Ad);
    }
    free(Bd);
}

/* Plain fp64 product of bf16 inputs, C[i][j] = sum_k A(i,k) B(j,k), with
 * arbitrary strides: the error-ablation reference and the exact product of
 * the backward identities dL/dx = dL/dy W, dL/dW = dL/dy^T x (Section 2.2). */
ORC_API void orc_gemm_bf16(const uint16_t *A, int64_t a_sr, int64_t a_sk,
                           const uint16_t *B, int64_t b_sr, int64_t b_sk,
                           int64_t K,
                           const int64_t *rows, int64_t n_rows, const int64_t *cols, int64_t n_cols,
                           double *C)
{
#pragma omp parallel for schedule(static)
    for (int64_t ii = 0; ii < n_rows; ++ii) {
        int64_t i = rows[ii];
        for (int64_t jj = 0; jj < n_cols; ++jj) {
            int64_t j = cols[jj];
            double s = 0.0;
            for (int64_t k = 0; k < K; ++k)
                s += bf16_to_double(A[i * a_sr + k * a_sk]) * bf16_to_double(B[j * b_sr + k * b_sk]);
            C[ii * n_cols + jj] = s;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Algorithm 3: MXFP4 linear-layer backward with the blockwise RHT            */
/* ------------------------------------------------------------------------- */

/* One operand view: transform (lines 3-6), then quantise (Algorithm 1 or 2).
 * Returns unpacked codes [R, K] and scales [R, K/32] (caller frees). */
ORC_API int orc_rht_quantize(const uint16_t *x, int64_t R, int64_t K, int64_t stride_r, int64_t stride_k,
                             int g, int rounding, uint64_t seed, uint32_t stream_tag,
                             float *y_out /* optional [R,K] */, uint8_t *codes, uint8_t *scales)
{
    float *y = y_out ? y_out : (float *)malloc((size_t)R * K * sizeof(float));
    if (!y) return -2;
    int rc = orc_rht(x, R, K, stride_r, stride_k, g, seed, y);
    if (rc == 0) rc = orc_quantize(y, R, K, rounding, seed, stream_tag, codes, scales);
    if (!y_out) free(y);
    return rc;
}

/* dY [b, m], X [b, n], W [m, n], all bf16 row-major.
 *   Q1 = Q(dY   blockdiag(S H))  [b, m]  groups along m   (stream_tag 1)
 *   Q2 = Q(W^T  blockdiag(S H))  [n, m]  groups along m   (stream_tag 2)
 *   Q3 = Q(dY^T blockdiag(S H))  [m, b]  groups along b   (stream_tag 3)
 *   Q4 = Q(X^T  blockdiag(S H))  [n, b]  groups along b   (stream_tag 4)
 *   dX = alpha Q1 Q2^T  [b, n];  dW = alpha Q3 Q4^T  [m, n];  alpha = 16/9 iff SR.
 * Only the sampled output rows/cols are produced (NULL = all). */
ORC_API int orc_linear_backward(const uint16_t *dY, const uint16_t *X, const uint16_t *W,
                                int64_t b, int64_t m, int64_t n, int g, int rounding, uint64_t seed,
                                const int64_t *dx_rows, int64_t n_dx_rows, const int64_t *dx_cols, int64_t n_dx_cols,
                                const int64_t *dw_rows, int64_t n_dw_rows, const int64_t *dw_cols, int64_t n_dw_cols,
                                double *dX, double *dW)
{
    const double alpha = (rounding != 1) ? 16.0 / 9.0 : 1.0;      /* both SR readings carry the 3/4 pre-scale */
    int rc = 0;
    uint8_t *c1 = (uint8_t *)malloc((size_t)b * m), *s1 = (uint8_t *)malloc((size_t)b * m / 32);
    uint8_t *c2 = (uint8_t *)malloc((size_t)n * m), *s2 = (uint8_t *)malloc((size_t)n * m / 32);
    rc |= orc_rht_quantize(dY, b, m, m, 1, g, rounding, seed, 1u, NULL, c1, s1);
    rc |= orc_rht_quantize(W, n, m, 1, n, g, rounding, seed, 2u, NULL, c2, s2);
    if (rc == 0)
        orc_gemm(c1, s1, c2, s2, b, n, m, alpha, dx_rows, n_dx_rows, dx_cols, n_dx_cols, dX);
    free(c1); free(s1); free(c2); free(s2);
    if (rc) return rc;
    uint8_t *c3 = (uint8_t *)malloc((size_t)m * b), *s3 = (uint8_t *)malloc((size_t)m * b / 32);
    uint8_t *c4 = (uint8_t *)malloc((size_t)n * b), *s4 = (uint8_t *)malloc((size_t)n * b / 32);
    rc |= orc_rht_quantize(dY, m, b, 1, m, g, rounding, seed, 3u, NULL, c3, s3);
    rc |= orc_rht_quantize(X, n, b, 1, n, g, rounding, seed, 4u, NULL, c4, s4);
    if (rc == 0)
        orc_gemm(c3, s3, c4, s4, m, n, b, alpha, dw_rows, n_dw_rows, dw_cols, n_dw_cols, dW);
    free(c3); free(s3); free(c4); free(s4);
    return rc;
}

/* Bias gradient of the linear layer y = x W^T + b (problem statement, Section 2: dL/db = 1 dL/dy): the column sums
 * of dY [b, m], computed exactly as a plain loop in fp64 (bf16 inputs are exact in fp64; 2^14 terms lose nothing
 * that matters).  Not quantised: the paper's recipe touches only the two matrix products. */
ORC_API void orc_bias_grad(const uint16_t *dY, int64_t b, int64_t m, double *db)
{
    for (int64_t j = 0; j < m; ++j) {
        double s = 0.0;
        for (int64_t i = 0; i < b; ++i) s += bf16_to_double(dY[i * m + j]);
        db[j] = s;
    }
}

ORC_API int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ========================================================================= */
/* Extensions beyond Algorithms 1-3 (each restates a remark of the paper)     */
/* ========================================================================= */

/* ------------------------------------------------------------------------- */
/* FP8 (E4M3) forward pass (Section 4.1, last remark; supplementary section   */
/* "FP8 Forward Pass Results"): y = x W^T with both operands quantised to     */
/* E4M3 under one scale per tensor, the product accumulated in high precision. */
/* The paper names the format and the library it used, not the arithmetic;     */
/* the reading here: scale = 448 / amax of the tensor (fp32 division; 1 for an */
/* all-zero tensor), element = round-to-nearest-even of fp32(x * scale) onto   */
/* the E4M3 grid, saturating at +-448, output = sum / (scale_x scale_w).       */
/* ------------------------------------------------------------------------- */

/* E4M3 ("fn": no infinities): 1 sign, 4 exponent (bias 7), 3 mantissa bits.  Exponent field 0 holds the subnormals
 * m/8 * 2^-6; exponent field 15 with mantissa 7 is NaN, so the largest value is 1.75 * 2^8 = 448. */
ORC_API double orc_e4m3_value(uint32_t code)
{
    uint32_t e = (code >> 3) & 15u, m = code & 7u;
    double v;
    if (e == 15u && m == 7u) return NAN;
    if (e == 0u) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, (int)e - 7);
    return (code & 0x80u) ? -v : v;
}

/* Nearest E4M3 value of a finite v (ties to the code with even mantissa bit), saturating at +-448: found by walking
 * the enumerated grid of the 127 non-negative finite codes 0x00..0x7E, which is increasing in the code. */
ORC_API uint32_t orc_e4m3_round(float v)
{
    uint32_t sign = signbit(v) ? 0x80u : 0u;
    double a = fabs((double)v);
    if (!(a == a)) return 0x7Fu;
    if (a >= 448.0) return sign | 0x7Eu;
    uint32_t lo = 0;
    while (lo + 1 < 0x7Fu && orc_e4m3_value(lo + 1) <= a) ++lo;       /* value(lo) <= a < value(lo + 1) */
    double f = orc_e4m3_value(lo), c = orc_e4m3_value(lo + 1);
    uint32_t pick;
    if (a - f < c - a) pick = lo;
    else if (a - f > c - a) pick = lo + 1;
    else pick = (lo & 1u) ? lo + 1 : lo;                               /* tie: even code */
    return sign | pick;
}

/* Scale of a bf16 tensor [R, K] (strided): 448 / amax in fp32, 1 when the tensor is all zero. */
ORC_API float orc_fp8_tensor_scale(const uint16_t *x, int64_t R, int64_t K, int64_t stride_r, int64_t stride_k)
{
    float amax = 0.0f;
    for (int64_t r = 0; r < R; ++r)
        for (int64_t k = 0; k < K; ++k) {
            float a = (float)fabs(bf16_to_double(x[r * stride_r + k * stride_k]));
            if (a > amax) amax = a;
        }
    return amax > 0.0f ? 448.0f / amax : 1.0f;
}

/* codes[r][k] = E4M3(fp32(x[r][k] * scale)) */
ORC_API void orc_fp8_quantize(const uint16_t *x, int64_t R, int64_t K, int64_t stride_r, int64_t stride_k, float scale,
                              uint8_t *codes /* [R, K] */)
{
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r)
        for (int64_t k = 0; k < K; ++k) {
            volatile float v = (float)bf16_to_double(x[r * stride_r + k * stride_k]) * scale;   /* one fp32 rounding */
            codes[r * K + k] = (uint8_t)orc_e4m3_round(v);
        }
}

/* C[i][j] = alpha sum_k value(A[i][k]) value(B[j][k]) in fp64 on the selected rows / columns (NULL = all). */
ORC_API void orc_fp8_gemm(const uint8_t *A, const uint8_t *B, int64_t M, int64_t N, int64_t K, double alpha,
                          const int64_t *rows, int64_t n_rows, const int64_t *cols, int64_t n_cols, double *C)
{
    if (!rows) n_rows = M;
    if (!cols) n_cols = N;
#pragma omp parallel for schedule(static)
    for (int64_t ii = 0; ii < n_rows; ++ii) {
        int64_t i = rows ? rows[ii] : ii;
        for (int64_t jj = 0; jj < n_cols; ++jj) {
            int64_t j = cols ? cols[jj] : jj;
            double s = 0.0;
            for (int64_t k = 0; k < K; ++k) s += orc_e4m3_value(A[i * K + k]) * orc_e4m3_value(B[j * K + k]);
            C[ii * n_cols + jj] = alpha * s;
        }
    }
}

/* The forward pass y [b, m] = x [b, n] W [m, n]^T through E4M3, on the selected rows / columns of y. */
ORC_API void orc_linear_forward_fp8(const uint16_t *x, const uint16_t *W, int64_t b, int64_t n, int64_t m,
                                    const int64_t *rows, int64_t n_rows, const int64_t *cols, int64_t n_cols, double *y)
{
    float sx = orc_fp8_tensor_scale(x, b, n, n, 1), sw = orc_fp8_tensor_scale(W, m, n, n, 1);
    uint8_t *cx = (uint8_t *)malloc((size_t)b * n), *cw = (uint8_t *)malloc((size_t)m * n);
    orc_fp8_quantize(x, b, n, n, 1, sx, cx);
    orc_fp8_quantize(W, m, n, n, 1, sw, cw);
    orc_fp8_gemm(cx, cw, b, m, n, 1.0 / ((double)sx * (double)sw), rows, n_rows, cols, n_cols, y);
    free(cx); free(cw);
}

/* ------------------------------------------------------------------------- */
/* MXINT4 elements (Section 3, opening: "our analysis also applies to other    */
/* low precision datatypes such as MXINT4").  The paper gives no definition;   */
/* the reading here: an element is a 4-bit sign-magnitude integer q in          */
/* [-7, 7], 32 elements share an E8M0 scale X, the value is q X.  The largest  */
/* power of two among the elements is 4 = 2^2, so Algorithm 1's rule is the     */
/* MXFP4 one, shared_exp = floor(log2 amax) - 2 (amax / X in [4, 8), values in  */
/* (7, 8) clip under nearest rounding); Algorithm 2 pre-scales by 3/4           */
/* (|w| < 6 <= 7) and rounds stochastically on the UNIFORM integer grid, which  */
/* is Eq. 1-2 as printed.  The product of two such operands estimates 9/16 of   */
/* the true product, as for MXFP4.  Code byte: bit 3 = sign, bits 0-2 = |q|.    */
/* ------------------------------------------------------------------------- */

ORC_API double orc_int4_value(uint32_t code)
{
    double v = (double)(code & 7u);
    return (code & 8u) ? -v : v;
}

/* Eq. 1-2 with the dither delta = 1/2 - (r + 1/2)/256 in (-1/2, 1/2), r the 8-bit draw of the element (the draw of
 * the MXFP4 path): ceil iff x + delta >= floor(x) + 1/2, i.e. iff 256 frac >= r + 1/2. */
ORC_API uint32_t orc_int4_sr_round(double w, uint32_t r)
{
    uint32_t sign = signbit(w) ? 8u : 0u;
    double a = fabs(w);
    if (a >= 7.0) return sign | 7u;                       /* unreachable after the 3/4 pre-scale */
    double fl = floor(a), delta = 0.5 - ((double)r + 0.5) / 256.0;
    uint32_t q = (uint32_t)fl + ((a + delta >= fl + 0.5) ? 1u : 0u);
    return sign | q;
}

/* nearest integer, ties to even, saturating at 7 (Algorithm 1 line 4 for this element format) */
ORC_API uint32_t orc_int4_rn_round(double w)
{
    uint32_t sign = signbit(w) ? 8u : 0u;
    double a = fabs(w);
    if (a >= 7.0) return sign | 7u;
    double fl = floor(a), fr = a - fl;
    uint32_t q = (uint32_t)fl;
    if (fr > 0.5 || (fr == 0.5 && (q & 1u))) ++q;
    return sign | q;
}

/* Algorithm 2 (rounding 0) / Algorithm 1 (rounding 1) with MXINT4 elements on fp32 pre-quantisation values y [R, K];
 * row_ids as in orc_quantize_rows.  Scale bytes follow orc_e8m0_from_amax. */
ORC_API int orc_mxint4_quantize_rows(const float *y, int64_t R, int64_t K, int rounding, uint64_t seed, uint32_t stream_tag,
                                     const int64_t *row_ids, uint8_t *codes, uint8_t *scales)
{
    if (K % 32 != 0 || (rounding != 0 && rounding != 1)) return -1;
    const int64_t nblk = K / 32;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < R; ++r)
        for (int64_t b = 0; b < nblk; ++b) {
            const float *V = y + r * K + b * 32;
            float amax = 0.0f;
            int finite = 1;
            for (int i = 0; i < 32; ++i) {
                float av = fabsf(V[i]);
                if (!(av == av) || isinf(av)) finite = 0;
                if (av > amax) amax = av;
            }
            uint32_t byte = finite ? orc_e8m0_from_amax(amax) : 255u;
            scales[r * nblk + b] = (uint8_t)byte;
            if (byte == 255u) { memset(codes + r * K + b * 32, 0, 32); continue; }
            int shared_exp = (int)byte - 127;
            for (int i = 0; i < 32; ++i) {
                int64_t elem = (row_ids ? row_ids[r] : r) * K + b * 32 + i;
                if (rounding == 0)
                    codes[r * K + b * 32 + i] = (uint8_t)orc_int4_sr_round(ldexp(0.75 * (double)V[i], -shared_exp),
                                                                           orc_sr_draw(seed, stream_tag, (uint64_t)elem));
                else
                    codes[r * K + b * 32 + i] = (uint8_t)orc_int4_rn_round(ldexp((double)V[i], -shared_exp));
            }
        }
    return 0;
}

/* C[i][j] = alpha sum_k q_A X_A q_B X_B in fp64 (the MXFP4 GEMM with integer elements) */
ORC_API void orc_mxint4_gemm(const uint8_t *A_codes, const uint8_t *A_scales, const uint8_t *B_codes, const uint8_t *B_scales,
                             int64_t M, int64_t N, int64_t K, double alpha,
                             const int64_t *rows, int64_t n_rows, const int64_t *cols, int64_t n_cols, double *C)
{
    const int64_t nblk = K / 32;
    if (!rows) n_rows = M;
    if (!cols) n_cols = N;
#pragma omp parallel for schedule(static)
    for (int64_t ii = 0; ii < n_rows; ++ii) {
        int64_t i = rows ? rows[ii] : ii;
        for (int64_t jj = 0; jj < n_cols; ++jj) {
            int64_t j = cols ? cols[jj] : jj;
            double s = 0.0;
            for (int64_t k = 0; k < K; ++k)
                s += ldexp(orc_int4_value(A_codes[i * K + k]), (int)A_scales[i * nblk + k / 32] - 127) *
                     ldexp(orc_int4_value(B_codes[j * K + k]), (int)B_scales[j * nblk + k / 32] - 127);
            C[ii * n_cols + jj] = alpha * s;
        }
    }
}
