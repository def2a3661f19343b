/* Plain integer matrix product, the definition of the result (CPU oracle; test
 * infrastructure only, never linked into the CUDA library).
 *
 *   C[i][j] = sum_k (int64) A[i][k] * (int64) B[k][j]
 *
 * A is M x K row-major int8, B is K x N row-major int8, C is M x N row-major int64.
 * The loop nest is the definition with the j loop innermost; rows of C are spread over
 * OpenMP threads when the file is built with -fopenmp.  No blocking, no intrinsics.
 * The residue variant reduces the same sum to the symmetric range of m afterwards. */
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_matmul_i64(const int8_t* A, const int8_t* B, int64_t* C, int64_t M, int64_t N, int64_t K)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < M; ++i) {
        int64_t* c = C + i * N;
        memset(c, 0, (size_t)N * sizeof(int64_t));
        for (int64_t k = 0; k < K; ++k) {
            const int64_t a = A[i * K + k];
            const int8_t* b = B + k * N;
            for (int64_t j = 0; j < N; ++j) c[j] += a * (int64_t)b[j];
        }
    }
}

/* The same definition in its textbook order (i, j, k innermost), on one thread: every entry is one
 * dot product of a row of A with a column of B.  Timed by the benchmark at 1024^3 as the naive
 * CPU reference point; also a second, independently ordered check of the loop nest above. */
void oracle_matmul_i64_ijk(const int8_t* A, const int8_t* B, int64_t* C, int64_t M, int64_t N, int64_t K)
{
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            int64_t acc = 0;
            for (int64_t k = 0; k < K; ++k) acc += (int64_t)A[i * K + k] * (int64_t)B[k * N + j];
            C[i * N + j] = acc;
        }
}

/* Rows i0 <= i < i1 only (for sampled checks at sizes where the whole product is too slow). */
void oracle_matmul_i64_rows(const int8_t* A, const int8_t* B, int64_t* C_rows, int64_t i0, int64_t i1,
                            int64_t N, int64_t K)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = i0; i < i1; ++i) {
        int64_t* c = C_rows + (i - i0) * N;
        memset(c, 0, (size_t)N * sizeof(int64_t));
        for (int64_t k = 0; k < K; ++k) {
            const int64_t a = A[i * K + k];
            const int8_t* b = B + k * N;
            for (int64_t j = 0; j < N; ++j) c[j] += a * (int64_t)b[j];
        }
    }
}

/* Symmetric residue of every entry: result in [-floor(m/2), ceil(m/2) - 1]. */
void oracle_mod_symmetric(int64_t* C, int64_t count, int64_t m)
{
    const int64_t lo = -(m / 2);
    for (int64_t t = 0; t < count; ++t) {
        int64_t x = (C[t] - lo) % m;
        if (x < 0) x += m;
        C[t] = x + lo;
    }
}

/* The same definition for 16-bit inputs (the width-12 significand products). */
void oracle_matmul_i64_s16_rows(const int16_t* A, const int16_t* B, int64_t* C_rows, int64_t i0, int64_t i1, int64_t N,
                                int64_t K)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = i0; i < i1; ++i) {
        int64_t* c = C_rows + (i - i0) * N;
        memset(c, 0, (size_t)N * sizeof(int64_t));
        for (int64_t k = 0; k < K; ++k) {
            const int64_t a = A[i * K + k];
            const int16_t* b = B + k * N;
            for (int64_t j = 0; j < N; ++j) c[j] += a * (int64_t)b[j];
        }
    }
}
