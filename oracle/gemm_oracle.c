/* GEMM oracle (TEST INFRASTRUCTURE -- shares nothing with the CUDA library).
 *
 * The swizzle of the paper's GEMM case study only changes WHICH block computes
 * which output tile; the product itself is the textbook one:
 *
 *     C[i][j] = sum_{k=0}^{K-1} A[i][k] * B[k][j]          (C is M x N, A is M x K, B is K x N)
 *
 * so the oracle is that definition written out: one fp64 accumulator per output
 * element, k ascending, no blocking, no reassociation, no fast-math.  Inputs are the
 * bf16 bit patterns the GPU receives, widened exactly (bf16 -> fp32 -> fp64 is exact;
 * a product of two bf16 values has at most 16 significant bits and is exact in fp64).
 * Beside the reference value it returns S[i][j] = sum_k |A[i][k]| * |B[k][j]|, the
 * scale the rounding noise of any fp32 accumulation is proportional to.
 *
 * Loop order is i-k-j: for a fixed output row the inner loop runs along j over
 * independent accumulators, so the compiler may vectorise it without changing any
 * sum's order.  OpenMP splits the list of requested rows across threads; each row is
 * computed by exactly one thread.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline float bf16_to_f32(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

int sp_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Widen a bf16 array to fp32 (exact). */
void sp_oracle_widen(const uint16_t* src, float* dst, int64_t n) {
    for (int64_t i = 0; i < n; ++i) dst[i] = bf16_to_f32(src[i]);
}

/* Rows `rows[0..nrows)` of C = A * B, columns [c0, c1).
 *   A: M x K row-major bf16 bits.
 *   B: b_is_nk == 0 -> K x N row-major (element (k,j) at B[k*N + j]);
 *      b_is_nk == 1 -> N x K row-major (element (k,j) at B[j*K + k]).
 *   ref, S: nrows x (c1 - c0) row-major fp64 outputs (S may be NULL).
 * Returns 0, or -1 on a bad argument / allocation failure. */
int sp_oracle_gemm_rows(const uint16_t* A, const uint16_t* B, int64_t M, int64_t N, int64_t K,
                        int b_is_nk, const int64_t* rows, int64_t nrows, int64_t c0, int64_t c1,
                        double* ref, double* S, int nthreads) {
    if (!A || !B || !ref || M <= 0 || N <= 0 || K <= 0 || nrows < 0 || c0 < 0 || c1 > N || c0 > c1) return -1;
    for (int64_t r = 0; r < nrows; ++r)
        if (rows[r] < 0 || rows[r] >= M) return -1;
    const int64_t W = c1 - c0;
    if (W == 0 || nrows == 0) return 0;

    /* B widened once to fp32, as a K x W panel with j contiguous (exact; only a layout copy). */
    float* Bw = (float*)malloc((size_t)K * (size_t)W * sizeof(float));
    if (!Bw) return -1;
    for (int64_t k = 0; k < K; ++k)
        for (int64_t j = 0; j < W; ++j)
            Bw[k * W + j] = b_is_nk ? bf16_to_f32(B[(c0 + j) * K + k]) : bf16_to_f32(B[k * N + (c0 + j)]);

#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < nrows; ++r) {
        const int64_t i = rows[r];
        double* acc = ref + r * W;
        double* sab = S ? S + r * W : NULL;
        for (int64_t j = 0; j < W; ++j) acc[j] = 0.0;
        if (sab) for (int64_t j = 0; j < W; ++j) sab[j] = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            const double a = (double)bf16_to_f32(A[i * K + k]);
            const double aa = fabs(a);
            const float* brow = Bw + k * W;
            for (int64_t j = 0; j < W; ++j) acc[j] += a * (double)brow[j];
            if (sab) for (int64_t j = 0; j < W; ++j) sab[j] += aa * fabs((double)brow[j]);
        }
    }
    free(Bw);
    return 0;
}
