/*
 * TEST INFRASTRUCTURE ONLY: the textbook triple loop, C[i,j] = sum_k A[i,k] * B[k,j]
 * (granular-operation table, Section 5: matmul(x, y) = sum(mul(x[i,k], y[k,j]), dim=k)),
 * on fp64 arrays, one scalar at a time, k ascending.  It is a separate translation unit
 * with no code in common with gmlp_oracle.c; the tests compose it with numpy to pin the
 * oracle's matmul stages on tiny shapes.
 */
#include <stdint.h>

void naive_matmul_f64(const double* A, const double* B, double* C, int64_t M, int64_t K, int64_t N)
{
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            double s = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                s += A[i * K + k] * B[k * N + j];
            }
            C[i * N + j] = s;
        }
    }
}
