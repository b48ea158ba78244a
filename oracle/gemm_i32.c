/* CPU oracle, integer GEMM of the W4A4 layer.  TEST INFRASTRUCTURE ONLY:
 * nothing in the CUDA library includes, links or calls this file.
 *
 * acc[m][n] = sum_k xq[m][k] * wq[n][k]   (Eq. 2's product, on the integer
 * codes of Eq. 1), the plain triple loop.  Each sum is carried in 64 bits and
 * must fit 32 bits; the only liberty taken is that the rows of the output are
 * shared among the host threads.
 */
#include <stdint.h>
#include <omp.h>

int oracle_gemm_threads(void) { return omp_get_max_threads(); }

/* xq: [M][K] int8, wq: [N][K] int8, acc: [M][N] int32.  Returns 0, or 1 if
 * any sum left the int32 range (acc then holds the truncated value). */
int oracle_gemm_i32(const int8_t* xq, int64_t M, const int8_t* wq, int64_t N,
                    int64_t K, int32_t* acc)
{
    int overflow = 0;
#pragma omp parallel for schedule(static) reduction(|:overflow)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            int64_t sum = 0;
            for (int64_t k = 0; k < K; ++k)
                sum += (int64_t)xq[m * K + k] * (int64_t)wq[n * K + k];
            if (sum > INT32_MAX || sum < INT32_MIN) overflow = 1;
            acc[m * N + n] = (int32_t)sum;
        }
    }
    return overflow;
}
