/*
 * CPU oracle for mixed-precision integer (MIP) GEMM and convolution.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct
 * statement of what the GPU library must compute.  It shares no code, header,
 * table or helper with the CUDA path and must never be linked into, imported
 * by or called from the product library; only the test-suite, the smoke check
 * and the benchmark's cpu-baseline / reference legs use it.
 *
 * What is computed (paper, Section 5 opening: INT8 products accumulated in
 * INT32; Section 7.3: C^q = A^q * B^q; Figure 1: the macro-kernel computes
 * C += A * B):
 *
 *   R(i,j) = (accumulate ? C_in(i,j) : 0) + sum_{k<K} a(i,k) * b(k,j)
 *
 * evaluated in 64-bit integers, a(i,k) sign-extended (int8) or zero-extended
 * (uint8), b(k,j) sign-extended (or, through mip_oracle_gemm_ex, zero-extended),
 * and then required to fit int32.  A cell whose
 * exact value does not fit is counted as an overflow cell (the result there is
 * the low 32 bits, and callers treat the configuration as invalid).
 *
 * Layouts: A row-major M x K (a(i,k) = A[i*lda + k]); B column-major K x N
 * (b(k,j) = B[j*ldb + k]); C row-major M x N (C[i*ldc + j]).  Padding columns
 * of C (j >= N) are never touched.
 *
 * Convolution (paper, Section 7.2, O = Conv(F, I)): direct seven-loop form on
 * channel-last tensors, never via im2col, so that it shares no structure with
 * the GPU's lowering:
 *
 *   Y[n][ho][wo][co] = sum_{r,s,c} X[n][ho*sh - ph + r*dh][wo*sw - pw + s*dw][c]
 *                                  * W[co][r][s][c]
 *
 * where a term whose input row or column falls outside the image contributes 0.
 *
 * Dequantised results: mip_oracle_dequant (definition C^r = s * C^q in binary64).
 * Requantised 8-bit codes: mip_oracle_requant (binary32 rule stated at the function).
 *
 * Pins: tests/test_oracle_pins.py (brute force on tiny inputs, closed forms,
 * extremes, range check, checksum identities, NumPy integer matmul, conv vs
 * explicit im2col, shifted-copy filters).
 */
#include <stdint.h>
#include <stddef.h>

static inline int64_t widen_a(const void *A, int64_t idx, int a_unsigned)
{
    if (a_unsigned)
        return (int64_t)((const uint8_t *)A)[idx];
    return (int64_t)((const int8_t *)A)[idx];
}

/*
 * Returns the number of overflow cells (0 = every cell fits int32), or -1 on
 * invalid arguments.
 */
int64_t mip_oracle_gemm_ex(int a_unsigned, int b_unsigned, int64_t M, int64_t N, int64_t K,
                           const void *A, int64_t lda,
                           const void *B, int64_t ldb,
                           int32_t *C, int64_t ldc, int accumulate)
{
    if (M < 0 || N < 0 || K < 0)
        return -1;
    if (M == 0 || N == 0)
        return 0;
    if (lda < K || ldb < K || ldc < N)
        return -1;
    if (!C || (K > 0 && (!A || !B)))
        return -1;

    int64_t overflow_cells = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow_cells)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            int64_t S = 0;
            for (int64_t k = 0; k < K; ++k) {
                int64_t a = widen_a(A, i * lda + k, a_unsigned);
                int64_t b = widen_a(B, j * ldb + k, b_unsigned);
                S += a * b;
            }
            int64_t R = (accumulate ? (int64_t)C[i * ldc + j] : 0) + S;
            if (R < (int64_t)INT32_MIN || R > (int64_t)INT32_MAX)
                overflow_cells += 1;
            C[i * ldc + j] = (int32_t)(uint32_t)(uint64_t)R;
        }
    }
    return overflow_cells;
}

/* The common case: B signed. */
int64_t mip_oracle_gemm(int a_unsigned, int64_t M, int64_t N, int64_t K,
                        const void *A, int64_t lda,
                        const int8_t *B, int64_t ldb,
                        int32_t *C, int64_t ldc, int accumulate)
{
    return mip_oracle_gemm_ex(a_unsigned, 0, M, N, K, A, lda, B, ldb, C, ldc, accumulate);
}

/*
 * Direct convolution, uint8 activations (zero-extended) x int8 filters
 * (sign-extended) -> int32.  X: [Nb][H][W][Cin]; Wt: [Cout][R][S][Cin];
 * Y: [Nb][Ho][Wo][Cout] with Ho = (H + 2*ph - dh*(R-1) - 1)/sh + 1 (same in w).
 * Returns overflow-cell count, or -1 on invalid arguments.
 */
int64_t mip_oracle_conv(int64_t Nb, int64_t H, int64_t W, int64_t Cin, int64_t Cout,
                        int64_t R, int64_t S,
                        int64_t sh, int64_t sw, int64_t ph, int64_t pw,
                        int64_t dh, int64_t dw,
                        const uint8_t *X, const int8_t *Wt, int32_t *Y, int accumulate)
{
    if (Nb < 0 || H <= 0 || W <= 0 || Cin <= 0 || Cout < 0 || R <= 0 || S <= 0)
        return -1;
    if (sh <= 0 || sw <= 0 || dh <= 0 || dw <= 0 || ph < 0 || pw < 0)
        return -1;
    int64_t eh = H + 2 * ph - dh * (R - 1) - 1;
    int64_t ew = W + 2 * pw - dw * (S - 1) - 1;
    if (eh < 0 || ew < 0)
        return -1;
    int64_t Ho = eh / sh + 1;
    int64_t Wo = ew / sw + 1;
    if (Nb == 0 || Cout == 0)
        return 0;
    if (!X || !Wt || !Y)
        return -1;

    int64_t overflow_cells = 0;
#pragma omp parallel for collapse(2) schedule(static) reduction(+ : overflow_cells)
    for (int64_t n = 0; n < Nb; ++n) {
        for (int64_t ho = 0; ho < Ho; ++ho) {
            for (int64_t wo = 0; wo < Wo; ++wo) {
                for (int64_t co = 0; co < Cout; ++co) {
                    int64_t acc = 0;
                    for (int64_t r = 0; r < R; ++r) {
                        int64_t h = ho * sh - ph + r * dh;
                        if (h < 0 || h >= H)
                            continue;
                        for (int64_t s = 0; s < S; ++s) {
                            int64_t w = wo * sw - pw + s * dw;
                            if (w < 0 || w >= W)
                                continue;
                            const uint8_t *x = X + ((n * H + h) * W + w) * Cin;
                            const int8_t *f = Wt + ((co * R + r) * S + s) * Cin;
                            for (int64_t c = 0; c < Cin; ++c)
                                acc += (int64_t)x[c] * (int64_t)f[c];
                        }
                    }
                    int64_t yi = ((n * Ho + ho) * Wo + wo) * Cout + co;
                    int64_t Rv = (accumulate ? (int64_t)Y[yi] : 0) + acc;
                    if (Rv < (int64_t)INT32_MIN || Rv > (int64_t)INT32_MAX)
                        overflow_cells += 1;
                    Y[yi] = (int32_t)(uint32_t)(uint64_t)Rv;
                }
            }
        }
    }
    return overflow_cells;
}

/*
 * Dequantisation of an integer result (paper, Section 7.3: C^r = s_A s_B C^q): every exact integer
 * sum is multiplied by the scale as a real number, here in binary64 (the product of a 32-bit
 * integer and a binary32 scale is exact in binary64: 31 + 24 significant bits).  The GPU path
 * rounds to binary32 twice (conversion, multiplication); tests allow the 2^-23 relative error
 * that follows from that.
 */
void mip_oracle_dequant(const int32_t *Cq, int64_t count, double scale, double *Cr)
{
    for (int64_t i = 0; i < count; ++i)
        Cr[i] = scale * (double)Cq[i];
}

/*
 * Requantisation of an integer result to 8-bit codes (the step that would follow C^q when the next
 * layer consumes integers again; the paper's scale-only scheme, Section 7.3, read backwards:
 * code = round(scale * C^q), saturated).  The paper fixes neither rounding nor precision.  Because
 * floating point decides an integer here, the rule is stated in the arithmetic the GPU epilogue uses,
 * binary32: t = fl32(fl32(sum) * scale), both roundings to nearest even; r = t rounded to the nearest
 * integer, ties to even; code = min(max(r, lo), hi).  `scale` must be finite.  Codes are returned as
 * int32 (the caller narrows them).  The pins check this rule against exact rational arithmetic.
 */
#include <math.h>
void mip_oracle_requant(const int32_t *Cq, int64_t count, float scale, int32_t lo, int32_t hi, int32_t *codes)
{
    for (int64_t i = 0; i < count; ++i) {
        volatile float as_float = (float)Cq[i];          /* (volatile: no wider intermediate) */
        volatile float t = as_float * scale;
        float r = rintf(t);                               /* default rounding mode: ties to even */
        if (r < (float)lo)
            r = (float)lo;
        if (r > (float)hi)
            r = (float)hi;
        codes[i] = (int32_t)r;
    }
}

/*
 * Per-output-channel integer bias, added to the exact integer sums before they are scaled (the usual
 * companion of the paper's scale-only scheme, Section 7.3: with the bias quantised at the scale
 * s_A s_B the real result is C^r = s_A s_B (C^q + b^q); the paper itself carries no bias, so this is
 * an extension).  out(i,j) = Cq(i,j) + bias[j], computed in int64 and range-checked into int32 like
 * every other sum here.  Cq and out are rows x cols, dense.  Returns the number of cells whose exact
 * value does not fit int32 (their low 32 bits are stored), or -1 on invalid arguments.
 */
int64_t mip_oracle_add_bias(const int32_t *Cq, int64_t rows, int64_t cols, const int32_t *bias, int32_t *out)
{
    if (rows < 0 || cols < 0 || (rows > 0 && cols > 0 && (!Cq || !bias || !out)))
        return -1;
    int64_t overflow_cells = 0;
    for (int64_t i = 0; i < rows; ++i) {
        for (int64_t j = 0; j < cols; ++j) {
            int64_t v = (int64_t)Cq[i * cols + j] + (int64_t)bias[j];
            if (v < (int64_t)INT32_MIN || v > (int64_t)INT32_MAX)
                overflow_cells += 1;
            out[i * cols + j] = (int32_t)(uint32_t)(uint64_t)v;
        }
    }
    return overflow_cells;
}

#ifdef _OPENMP
#include <omp.h>
int mip_oracle_threads(void) { return omp_get_max_threads(); }
#else
int mip_oracle_threads(void) { return 1; }
#endif
