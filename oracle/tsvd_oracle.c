/*
 * CPU checker for the Ternary-SVD linear map  y = U (diag(S) (V x)).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * GPU library is compared against; the library never calls it and shares no
 * code with it.  It works on the unpacked int8 ternary matrices and knows
 * nothing of any packed format.
 *
 * What it computes, in the paper's order of application (Section
 * "Truncated SVD in Network Compression", the display after Eq. 2, and the
 * cost table of the supplement, Table S1):
 *
 *   V-stage   zraw[k] = sum_n V[k,n] x[n]     additions/subtractions only,
 *                                             one per nonzero of V      (row "V(.)")
 *   S-stage   z[k]    = S[k] * zraw[k]        K multiplications         (row "diag(s)(.)")
 *   U-stage   y[m]    = sum_k U[m,k] z[k]     one add/sub per nonzero   (row "U(.)")
 *   bias      y[m]   += b[m]                  optional.  Eq. 1 is written "without any
 *                                             bias", yet every layer of the supplement's
 *                                             architecture listing has bias=True: the
 *                                             converted layer keeps the original layer's
 *                                             bias, one addition per output.
 *
 * Floating-point activations are accumulated in IEEE double in index order.
 * int8 activations take the V-stage in 64-bit integers (exact), then the
 * S- and U-stage in double.  S is single precision in storage and is widened
 * exactly.  Zero entries of U and V are skipped, never multiplied.
 *
 * Layout: U [M,K] row-major, V [K,N] row-major, x token-major (token b at
 * x + b*N), y token-major (token b at y + b*M), zraw token-major (b*K).
 *
 * Parity pins (tests/test_oracle_pins.py): dense reconstruction W' = U diag(S) V
 * on tiny shapes, exact integer evaluation, hand-worked 4x4 cases, the Winograd
 * F(2,3) and F(2x2,3x3) closed forms, linearity / sign / permutation invariants,
 * the operation counts of Table S1 and the plus/minus split of the Discussion.
 */
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int tsvd_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* returns 0, or 1 if an entry of U or V is outside {-1,0,+1}, or 2 on allocation failure */
static int check_ternary(const int8_t* A, long long n)
{
    for (long long i = 0; i < n; ++i)
        if (A[i] < -1 || A[i] > 1) return 1;
    return 0;
}

/*
 * counts (optional, length 2): counts[0] = additions+subtractions performed
 * (the bias additions included when there is a bias), counts[1] = multiplications
 * performed, summed over all B columns.  bias: NULL, or M single-precision values.
 */
int tsvd_oracle_forward_f64(const int8_t* U, const float* S, const int8_t* V,
                            int M, int K, int N,
                            const double* x, int B, const float* bias,
                            double* y, double* zraw_out, long long* counts)
{
    if (check_ternary(U, (long long)M * K) || check_ternary(V, (long long)K * N)) return 1;
    double* z = (double*)malloc(sizeof(double) * (size_t)B * (size_t)K + 8);
    if (!z) return 2;
    long long adds = 0, muls = 0;

    /* V-stage then S-stage */
#pragma omp parallel for collapse(2) reduction(+ : adds, muls) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int k = 0; k < K; ++k) {
            const int8_t* vrow = V + (size_t)k * N;
            const double* xb = x + (size_t)b * N;
            double acc = 0.0;
            for (int n = 0; n < N; ++n) {
                if (vrow[n] == 1) { acc += xb[n]; ++adds; }
                else if (vrow[n] == -1) { acc -= xb[n]; ++adds; }
            }
            if (zraw_out) zraw_out[(size_t)b * K + k] = acc;
            z[(size_t)b * K + k] = (double)S[k] * acc;
            ++muls;
        }
    }

    /* U-stage */
#pragma omp parallel for collapse(2) reduction(+ : adds) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int m = 0; m < M; ++m) {
            const int8_t* urow = U + (size_t)m * K;
            const double* zb = z + (size_t)b * K;
            double acc = 0.0;
            for (int k = 0; k < K; ++k) {
                if (urow[k] == 1) { acc += zb[k]; ++adds; }
                else if (urow[k] == -1) { acc -= zb[k]; ++adds; }
            }
            if (bias) { acc += (double)bias[m]; ++adds; }
            y[(size_t)b * M + m] = acc;
        }
    }
    free(z);
    if (counts) { counts[0] = adds; counts[1] = muls; }
    return 0;
}

/* int8 activations: zraw_out (optional) receives the exact integer V x as int64. */
int tsvd_oracle_forward_i8(const int8_t* U, const float* S, const int8_t* V,
                           int M, int K, int N,
                           const int8_t* x, int B, const float* bias,
                           double* y, long long* zraw_out, long long* counts)
{
    if (check_ternary(U, (long long)M * K) || check_ternary(V, (long long)K * N)) return 1;
    double* z = (double*)malloc(sizeof(double) * (size_t)B * (size_t)K + 8);
    if (!z) return 2;
    long long adds = 0, muls = 0;

#pragma omp parallel for collapse(2) reduction(+ : adds, muls) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int k = 0; k < K; ++k) {
            const int8_t* vrow = V + (size_t)k * N;
            const int8_t* xb = x + (size_t)b * N;
            long long acc = 0;
            for (int n = 0; n < N; ++n) {
                if (vrow[n] == 1) { acc += xb[n]; ++adds; }
                else if (vrow[n] == -1) { acc -= xb[n]; ++adds; }
            }
            if (zraw_out) zraw_out[(size_t)b * K + k] = acc;
            z[(size_t)b * K + k] = (double)S[k] * (double)acc;
            ++muls;
        }
    }

#pragma omp parallel for collapse(2) reduction(+ : adds) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int m = 0; m < M; ++m) {
            const int8_t* urow = U + (size_t)m * K;
            const double* zb = z + (size_t)b * K;
            double acc = 0.0;
            for (int k = 0; k < K; ++k) {
                if (urow[k] == 1) { acc += zb[k]; ++adds; }
                else if (urow[k] == -1) { acc -= zb[k]; ++adds; }
            }
            if (bias) { acc += (double)bias[m]; ++adds; }
            y[(size_t)b * M + m] = acc;
        }
    }
    free(z);
    if (counts) { counts[0] = adds; counts[1] = muls; }
    return 0;
}
