/*
 * CPU oracle for the stand-alone reductions.  TEST INFRASTRUCTURE ONLY: nothing in the
 * library or its binding includes, links or calls this file, and it shares no code with
 * the CUDA sources.
 *
 * Definitions (paper, Prompts appendix): task 14 "Reduction": the sum of all elements of
 * an fp32 array; task 15 "Dot Product": A.B = sum_{i=0}^{n-1} A_i * B_i; task 7 "Mean
 * Square Error": MSE = (1/N) sum_{i=1}^{N} (predictions_i - targets_i)^2.
 *
 * Each is the definition written out: one loop over i in ascending order, every term
 * formed and accumulated in fp64 (an fp32 value widens exactly; the product of two fp32
 * values is exact in fp64).  The second return value of each routine is sum_i |term_i|,
 * the scale against which the GPU result's rounding error is bounded.
 *
 * Parity: pinned by tests that do not go through this file (closed forms on integers,
 * exactly rounded summation, library fp64 routines).
 */
#include <math.h>
#include <stdint.h>

enum { ORACLE_REDUCE_SUM = 0, ORACLE_REDUCE_DOT = 1, ORACLE_REDUCE_MSE = 2 };

/* result[0] = the reduction, result[1] = sum of |terms| (before the 1/n of MSE). */
int oracle_reduce_f32(int kind, const float* x, const float* y, int64_t n, double* result) {
    if (!x || !result || n < 0 || (kind != ORACLE_REDUCE_SUM && !y)) return -1;
    double acc = 0.0, mag = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double term;
        if (kind == ORACLE_REDUCE_SUM) {
            term = (double)x[i];
        } else if (kind == ORACLE_REDUCE_DOT) {
            term = (double)x[i] * (double)y[i];
        } else if (kind == ORACLE_REDUCE_MSE) {
            const double d = (double)x[i] - (double)y[i];
            term = d * d;
        } else {
            return -1;
        }
        acc += term;
        mag += fabs(term);
    }
    result[0] = (kind == ORACLE_REDUCE_MSE && n > 0) ? acc / (double)n : acc;
    result[1] = mag;
    return 0;
}
