/*
 * TEST INFRASTRUCTURE - not part of the product path.
 *
 * Plain CPU fp64 GEMM that the GPU path is checked against.  The persistent GEMM
 * that the scheduler of Section 7.1.2 drives computes exactly C = A * B; the method
 * changes *where* each output tile is computed, never *what* is computed, so the
 * oracle is the textbook definition written out:
 *
 *     C[i][j] = sum_{k=0..K-1} (double)A[i][k] * (double)B[k][j]
 *
 * A is M x K, B is K x N, both row-major bf16 given as raw 16-bit patterns;
 * C is M x N row-major fp64.  The sum runs over k in ascending order.
 * A product of two bf16 values has at most 16 significant bits, so it is exact in
 * fp64 (fused or not); only the additions round.
 *
 * Only tests, the smoke check and the bench's cpu_baseline leg may call this.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_f64(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Triple loop, single thread: the definition itself. */
void oracle_gemm_bruteforce(const uint16_t* A, const uint16_t* B, double* C,
                            int64_t M, int64_t N, int64_t K) {
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            double s = 0.0;
            for (int64_t k = 0; k < K; ++k)
                s += bf16_to_f64(A[i * K + k]) * bf16_to_f64(B[k * N + j]);
            C[i * N + j] = s;
        }
}

/* One output entry (used for sampled checks at sizes where a full C is too slow). */
double oracle_gemm_entry(const uint16_t* A, const uint16_t* B,
                         int64_t N, int64_t K, int64_t i, int64_t j) {
    double s = 0.0;
    for (int64_t k = 0; k < K; ++k)
        s += bf16_to_f64(A[i * K + k]) * bf16_to_f64(B[k * N + j]);
    return s;
}

/* Rows [row0,row1) x columns [col0,col1) of C, written densely into
 * out[(row1-row0) x (col1-col0)].  Row panels are spread over OpenMP threads;
 * every output still adds its K terms in ascending k, so the result equals the
 * brute-force loop bit for bit. */
void oracle_gemm_block(const uint16_t* A, const uint16_t* B, double* out,
                       int64_t M, int64_t N, int64_t K,
                       int64_t row0, int64_t row1, int64_t col0, int64_t col1) {
    (void)M;
    const int64_t nc = col1 - col0, nr = row1 - row0;
    if (nc <= 0 || nr <= 0) return;
    double* Bd = (double*)malloc(sizeof(double) * (size_t)K * (size_t)nc);
    #pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < K; ++k)
        for (int64_t j = 0; j < nc; ++j)
            Bd[k * nc + j] = bf16_to_f64(B[k * N + col0 + j]);
    const int64_t JB = 512;   /* column block: 4 KB of C per row stays in L1 */
    #pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < nr; ++i) {
        double* c = out + i * nc;
        const uint16_t* a = A + (row0 + i) * K;
        for (int64_t j0 = 0; j0 < nc; j0 += JB) {
            const int64_t j1 = j0 + JB < nc ? j0 + JB : nc;
            for (int64_t j = j0; j < j1; ++j) c[j] = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                const double av = bf16_to_f64(a[k]);
                const double* b = Bd + k * nc;
                for (int64_t j = j0; j < j1; ++j) c[j] += av * b[j];
            }
        }
    }
    free(Bd);
}

void oracle_gemm_blocked(const uint16_t* A, const uint16_t* B, double* C,
                         int64_t M, int64_t N, int64_t K) {
    oracle_gemm_block(A, B, C, M, N, K, 0, M, 0, N);
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
