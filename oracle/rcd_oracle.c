/*
 * CPU oracle for the resource-constrained submodular data partition (RCD-SGD,
 * Algorithm 1 with the facility-location objective of Section 4, item 2).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, single-threaded
 * restatement of what the paper defines, used only to check the CUDA library
 * and to time a CPU baseline.  It shares no code, header, table or helper with
 * the CUDA library and nothing in the library calls it.
 *
 * Arithmetic: int8 features -> exact integer similarities and objective in
 * int64; bf16 features -> the bf16 bit patterns widened exactly to double and
 * everything summed in double, in ascending index order.
 *
 * Readings of the paper taken here (it is silent on each):
 *   - f(emptyset) = 0 and negative similarities never lower the value:
 *       f(A) = sum_{i in V_l} max(0, max_{v' in A} S[i][v'])
 *     (equal to the facility-location formula whenever S >= 0, as with the
 *     paper's Gaussian kernel; keeps f monotone submodular for dot products
 *     and cosines, which can be negative).
 *   - argmin over J (Algorithm 1) breaks ties toward the lowest j; GreedyStep's
 *     argmax breaks ties toward the lowest sample index inside the class.
 *   - C_{l,j} = |V_l| r_j / sum r is made an integer by largest-remainder
 *     apportionment (rcd_oracle_quotas below).
 *   - "exists v in R s.t. A u {v} in C_{l,j*}" is the cardinality test
 *     |A_{j*}| + 1 <= C_{l,j*}.
 *
 * Parity pins: every function below is pinned by tests/test_oracle_*.py
 * (closed forms, hand-worked traces, brute force on tiny inputs, invariants).
 * The actual assignments on the large synthetic workloads have no value printed
 * in the paper to compare with: for those the oracle is pinned only through
 * these properties.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

/* ------------------------------------------------------------------------- */
/* Similarity: S[a][b] = <x_a, x_b>  (Section 3.1: "similarities between each
 * data point are computed using vectors v, v'"; dot product / cosine).        */

void rcd_oracle_similarity_i8(const int8_t *X, int64_t M, int64_t d, int64_t *S)
{
    for (int64_t a = 0; a < M; ++a)
        for (int64_t b = 0; b < M; ++b) {
            int64_t acc = 0;
            for (int64_t k = 0; k < d; ++k)
                acc += (int64_t)X[a * d + k] * (int64_t)X[b * d + k];
            S[a * M + b] = acc;
        }
}

static double bf16_to_double(uint16_t bits)
{
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Rows are expected to be L2-normalised by the caller, so this is the cosine. */
void rcd_oracle_similarity_bf16(const uint16_t *Xbits, int64_t M, int64_t d, double *S)
{
    double *X = (double *)malloc((size_t)(M * d) * sizeof(double));
    for (int64_t i = 0; i < M * d; ++i) X[i] = bf16_to_double(Xbits[i]);
    for (int64_t a = 0; a < M; ++a)
        for (int64_t b = 0; b < M; ++b) {
            double acc = 0.0;
            for (int64_t k = 0; k < d; ++k)
                acc += X[a * d + k] * X[b * d + k];
            S[a * M + b] = acc;
        }
    free(X);
}

/* Gaussian-kernel similarity (Section 4, item 2: "a Gaussian kernel with L2 distance",
 * bandwidth sigma = sum_{v,v'} ||v - v'||_2 / n^2).  The paper gives neither the exponent
 * nor what n counts; the reading taken here: n = |V_l| (the class), the sum runs over all
 * ordered pairs (the zero diagonal included), and
 *     sim(v, v') = exp(-||v - v'||^2 / (2 sigma^2)).
 * A class whose points all coincide has sigma = 0; every similarity is then 1.
 * X holds the features already widened to double; S and *sigma_out are outputs.           */
static void gaussian_from_doubles(const double *X, int64_t M, int64_t d, double *S, double *sigma_out)
{
    double total = 0.0;
    for (int64_t a = 0; a < M; ++a)
        for (int64_t b = 0; b < M; ++b) {
            double sq = 0.0;
            for (int64_t k = 0; k < d; ++k) {
                double diff = X[a * d + k] - X[b * d + k];
                sq += diff * diff;
            }
            S[a * M + b] = sq;                  /* squared distance for now */
            total += sqrt(sq);
        }
    double sigma = M > 0 ? total / ((double)M * (double)M) : 0.0;
    for (int64_t i = 0; i < M * M; ++i)
        S[i] = sigma > 0.0 ? exp(-S[i] / (2.0 * sigma * sigma)) : 1.0;
    if (sigma_out) *sigma_out = sigma;
}

void rcd_oracle_gaussian_i8(const int8_t *X, int64_t M, int64_t d, double *S, double *sigma_out)
{
    double *Xd = (double *)malloc((size_t)(M * d + 1) * sizeof(double));
    for (int64_t i = 0; i < M * d; ++i) Xd[i] = (double)X[i];
    gaussian_from_doubles(Xd, M, d, S, sigma_out);
    free(Xd);
}

void rcd_oracle_gaussian_bf16(const uint16_t *Xbits, int64_t M, int64_t d, double *S, double *sigma_out)
{
    double *Xd = (double *)malloc((size_t)(M * d + 1) * sizeof(double));
    for (int64_t i = 0; i < M * d; ++i) Xd[i] = bf16_to_double(Xbits[i]);
    gaussian_from_doubles(Xd, M, d, S, sigma_out);
    free(Xd);
}

/* ------------------------------------------------------------------------- */
/* Quotas (Algorithm 1, "Constraint C_{l,j} = |V_l| r_j / sum_j r_j").
 * Largest-remainder rule: floor every share, then hand the left-over units one
 * each to the largest fractional parts, ties toward the lowest j.             */

void rcd_oracle_quotas(int64_t M, const double *r, int32_t W, int32_t *C)
{
    volatile double R = 0.0;            /* volatile: no contraction / reassociation */
    for (int32_t j = 0; j < W; ++j) R = R + r[j];
    double *frac = (double *)malloc((size_t)W * sizeof(double));
    int64_t given = 0;
    for (int32_t j = 0; j < W; ++j) {
        volatile double num = (double)M * r[j];
        volatile double q = num / R;
        double fl = floor(q);
        C[j] = (int32_t)fl;
        frac[j] = q - fl;
        given += C[j];
    }
    int64_t left = M - given;
    while (left > 0) {                  /* left < W: one extra unit per chosen worker */
        int32_t best = -1;
        for (int32_t j = 0; j < W; ++j)
            if (frac[j] >= 0.0 && (best < 0 || frac[j] > frac[best])) best = j;
        C[best] += 1;
        frac[best] = -1.0;
        left -= 1;
    }
    while (left < 0) {                  /* only if rounding pushed a share up to the next integer */
        int32_t worst = -1;
        for (int32_t j = 0; j < W; ++j)
            if (C[j] > 0 && frac[j] >= 0.0 && (worst < 0 || frac[j] <= frac[worst])) worst = j;
        C[worst] -= 1;
        frac[worst] = -1.0;
        left += 1;
    }
    free(frac);
}

/* ------------------------------------------------------------------------- */
/* The typed part: objective, Algorithm 1 (plain and incremental), replay.     */

#define VT int64_t
#define SUF(name) name##_i64
#include "rcd_oracle_typed.inc"
#undef VT
#undef SUF

#define VT double
#define SUF(name) name##_f64
#include "rcd_oracle_typed.inc"
#undef VT
#undef SUF
