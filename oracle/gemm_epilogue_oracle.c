/*
 * CPU oracle for Y = act(A.B + bias).  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the GPU library is checked
 * against.  It is not part of the product path: nothing in the library or its
 * Python binding includes, links or calls it, and it shares no code, header,
 * table or constant with the CUDA sources.
 *
 * What it computes (paper, Prompts appendix, task 2 "Matrix Multiplication":
 * A is M x K, B is K x N, C = A x B is M x N; matmul case study, "Common
 * setup": all matrices row-major, element (r, c) of an R x C matrix at
 * index r*C + c; Prompts appendix, task 10: ReLU(x) = max(0, x)):
 *
 *   y_ref[m][n] = act( sum_{k=0..K-1} (double)A[m][k] * (double)B[k][n]
 *                      + (double)bias[n] )
 *
 * The sum runs over k in ascending order in fp64; act is evaluated in fp64.
 * Inputs are fp32 values or bf16 bit patterns; both widen to fp64 exactly, and
 * every product of two such values is exact in fp64, so the only rounding is
 * in the running sum.  The bias vector (length N, broadcast over rows) and the
 * tanh form of GELU are not in the paper; they follow this project's problem
 * statement:
 *
 *   GELU_tanh(x) = 0.5 x (1 + tanh( sqrt(2/pi) (x + 0.044715 x^3) ))
 *
 * act = sigmoid is 1 / (1 + exp(-x)) (Prompts appendix, task 1).
 *
 * The loop nest is the plain triple loop in i-k-j order (row, reduction index,
 * column) with one fp64 accumulator per output column; rows are dealt to host
 * threads.  No blocking, no vector intrinsics, no reordering of the k sum.
 *
 * Output rounding helpers (double -> fp32, double -> bf16, both
 * round-to-nearest-even, written here at bit level) serve the bit-exact checks
 * on integer-valued cases.
 *
 * Parity: every function here is pinned by tests that do not go through this
 * file (closed forms, exact integer arithmetic, library fp64 routines).
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1 };
enum { ORACLE_ACT_NONE = 0, ORACLE_ACT_RELU = 1, ORACLE_ACT_GELU_TANH = 2, ORACLE_ACT_SIGMOID = 3 };

/* bf16 is the upper half of an IEEE fp32: widening is a 16-bit shift. */
double oracle_bf16_to_double(uint16_t bits) {
    uint32_t w = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* double -> bf16, one rounding, ties to even.  Works on the fp64 bit pattern:
 * bf16 keeps 8 exponent bits (bias 127) and 7 fraction bits. */
uint16_t oracle_bf16_from_double(double x) {
    uint64_t u;
    memcpy(&u, &x, sizeof u);
    uint16_t sign = (uint16_t)((u >> 63) << 15);
    int64_t e = (int64_t)((u >> 52) & 0x7FF);
    uint64_t frac = u & 0xFFFFFFFFFFFFFull;
    if (e == 0x7FF) {                       /* inf or NaN */
        return (uint16_t)(sign | 0x7F80 | (frac ? 0x40 : 0));
    }
    if (e == 0) return sign;                /* fp64 zero / subnormal: far below bf16 range */
    int64_t eb = e - 1023 + 127;            /* bf16 biased exponent if normal */
    uint64_t sig = frac | (1ull << 52);     /* 53-bit significand, value sig * 2^(e-1075) */
    int shift = 52 - 7;                     /* bits to drop for a normal result */
    if (eb <= 0) {                          /* subnormal bf16: drop more bits */
        shift += (int)(1 - eb);
        eb = 0;
        if (shift > 62) return sign;        /* below half the smallest subnormal */
    }
    uint64_t kept = sig >> shift;
    uint64_t rem = sig & ((1ull << shift) - 1);
    uint64_t half = 1ull << (shift - 1);
    if (rem > half || (rem == half && (kept & 1))) kept += 1;
    /* kept holds the hidden bit (normal) or not (subnormal); adding it to the
     * exponent field makes a mantissa carry bump the exponent by itself. */
    uint64_t out = (eb == 0) ? kept : (((uint64_t)(eb - 1) << 7) + kept);
    if (out >= 0x7F80) out = 0x7F80;        /* overflow to infinity */
    return (uint16_t)(sign | (uint16_t)out);
}

/* double -> fp32: the C conversion rounds to nearest even in the default mode. */
float oracle_f32_from_double(double x) { return (float)x; }

double oracle_act(double x, int act) {
    switch (act) {
    case ORACLE_ACT_RELU:
        return x > 0.0 ? x : 0.0;
    case ORACLE_ACT_GELU_TANH: {
        const double c = 0.7978845608028654; /* sqrt(2/pi) */
        return 0.5 * x * (1.0 + tanh(c * (x + 0.044715 * x * x * x)));
    }
    case ORACLE_ACT_SIGMOID:              /* Prompts appendix, task 1: 1 / (1 + exp(-x)) */
        return 1.0 / (1.0 + exp(-x));
    default:
        return x;
    }
}

static inline double load_elem(const void* p, int64_t i, int dtype) {
    if (dtype == ORACLE_F32) return (double)((const float*)p)[i];
    return oracle_bf16_to_double(((const uint16_t*)p)[i]);
}

typedef struct {
    const void *A, *B, *bias;
    double* y;
    int64_t M, N, K;
    int dtype, act;
    const int64_t *rows, *cols;   /* NULL = all */
    int64_t nrows, ncols;
    int64_t r0, r1;               /* slice of the (sampled) row list */
} job_t;

static void* run_rows(void* arg) {
    const job_t* j = (const job_t*)arg;
    const int64_t nc = j->cols ? j->ncols : j->N;
    for (int64_t ri = j->r0; ri < j->r1; ++ri) {
        const int64_t m = j->rows ? j->rows[ri] : ri;
        double* acc = j->y + ri * nc;
        for (int64_t c = 0; c < nc; ++c) acc[c] = 0.0;
        for (int64_t k = 0; k < j->K; ++k) {
            const double a = load_elem(j->A, m * j->K + k, j->dtype);
            for (int64_t c = 0; c < nc; ++c) {
                const int64_t n = j->cols ? j->cols[c] : c;
                acc[c] += a * load_elem(j->B, k * j->N + n, j->dtype);
            }
        }
        for (int64_t c = 0; c < nc; ++c) {
            const int64_t n = j->cols ? j->cols[c] : c;
            const double b = j->bias ? load_elem(j->bias, n, j->dtype) : 0.0;
            acc[c] = oracle_act(acc[c] + b, j->act);
        }
    }
    return NULL;
}

static int run(job_t base, int64_t nr, int nthreads) {
    if (nthreads < 1) nthreads = 1;
    if (nthreads > 256) nthreads = 256;
    if ((int64_t)nthreads > nr) nthreads = (int)(nr > 0 ? nr : 1);
    pthread_t tid[256];
    job_t jobs[256];
    for (int t = 0; t < nthreads; ++t) {
        jobs[t] = base;
        jobs[t].r0 = nr * t / nthreads;
        jobs[t].r1 = nr * (t + 1) / nthreads;
    }
    if (nthreads == 1) { run_rows(&jobs[0]); return 1; }
    for (int t = 0; t < nthreads; ++t)
        if (pthread_create(&tid[t], NULL, run_rows, &jobs[t]) != 0) return -1;
    for (int t = 0; t < nthreads; ++t) pthread_join(tid[t], NULL);
    return nthreads;
}

/* Full result: y_ref is M*N doubles, row-major.  bias may be NULL (zeros).
 * Returns the number of threads used, or -1. */
int oracle_gemm_epilogue(const void* A, const void* B, const void* bias, double* y_ref,
                         int64_t M, int64_t N, int64_t K, int dtype, int act, int nthreads) {
    if (!A || !B || !y_ref || M < 0 || N < 0 || K < 0) return -1;
    job_t j = {A, B, bias, y_ref, M, N, K, dtype, act, NULL, NULL, 0, 0, 0, 0};
    return run(j, M, nthreads);
}

/* Sampled result: y_ref[i*ncols + j] = y_ref at (rows[i], cols[j]); the same
 * loops as above restricted to the listed rows and columns. */
int oracle_gemm_epilogue_sampled(const void* A, const void* B, const void* bias, double* y_ref,
                                 int64_t M, int64_t N, int64_t K, int dtype, int act,
                                 const int64_t* rows, int64_t nrows,
                                 const int64_t* cols, int64_t ncols, int nthreads) {
    if (!A || !B || !y_ref || !rows || !cols) return -1;
    for (int64_t i = 0; i < nrows; ++i) if (rows[i] < 0 || rows[i] >= M) return -1;
    for (int64_t i = 0; i < ncols; ++i) if (cols[i] < 0 || cols[i] >= N) return -1;
    job_t j = {A, B, bias, y_ref, M, N, K, dtype, act, rows, cols, nrows, ncols, 0, 0};
    return run(j, nrows, nthreads);
}

/* Round n fp64 values to dtype (fp32 or bf16 bits), nearest-even; -0 -> +0 so
 * bit comparisons treat the two zeros alike. */
void oracle_round_to_dtype(const double* y, void* out, int64_t n, int dtype) {
    for (int64_t i = 0; i < n; ++i) {
        double v = y[i] == 0.0 ? 0.0 : y[i];
        if (dtype == ORACLE_F32) ((float*)out)[i] = oracle_f32_from_double(v);
        else ((uint16_t*)out)[i] = oracle_bf16_from_double(v);
    }
}
