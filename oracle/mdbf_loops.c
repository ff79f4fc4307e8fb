/*
 * Scalar-loop twin of oracle/mdbf_oracle.py.  TEST INFRASTRUCTURE ONLY: it is
 * never linked into, loaded by or called from the product library.
 *
 * Every entry of W_hat is written out from the element-wise statement of the
 * format (Eq. me-dbf-basis):
 *
 *   W_hat[n][i] = sum_j  ( S_A[n][j] * sum_t U_A[n][t] V_A[j][t] )
 *                      * ( S_B[j][i] * sum_s U_B[j][s] V_B[i][s] )
 *
 * with no blocking, no reordering and no library call, in double precision.
 * All matrices are dense row-major.  Signs are int8 (+1 / -1).
 *
 * Build:  gcc -O2 -shared -fPIC -o libmdbf_loops.so mdbf_loops.c
 */
#include <stdint.h>
#include <stddef.h>

static double envelope_entry(const double *U, const double *V, int r, int c, int l)
{
    double e = 0.0;
    for (int t = 0; t < l; ++t) e += U[(size_t)r * l + t] * V[(size_t)c * l + t];
    return e;
}

/* W: d_out x d_in, row-major.  Returns 0, or -1 on a sign that is not +-1. */
int mdbf_loops_reconstruct(const int8_t *S_A, const int8_t *S_B,
                           const double *U_A, const double *V_A,
                           const double *U_B, const double *V_B,
                           int d_out, int d_in, int k, int l, double *W)
{
    for (size_t e = 0; e < (size_t)d_out * k; ++e)
        if (S_A[e] != 1 && S_A[e] != -1) return -1;
    for (size_t e = 0; e < (size_t)k * d_in; ++e)
        if (S_B[e] != 1 && S_B[e] != -1) return -1;
    for (int n = 0; n < d_out; ++n) {
        for (int i = 0; i < d_in; ++i) {
            double w = 0.0;
            for (int j = 0; j < k; ++j) {
                double u_hat = (double)S_A[(size_t)n * k + j] * envelope_entry(U_A, V_A, n, j, l);
                double v_hat = (double)S_B[(size_t)j * d_in + i] * envelope_entry(U_B, V_B, j, i, l);
                w += u_hat * v_hat;
            }
            W[(size_t)n * d_in + i] = w;
        }
    }
    return 0;
}

/* X: d_in x T row-major, Y: d_out x T row-major.  Y = W_hat X by triple loop;
 * scratch W must hold d_out*d_in doubles. */
int mdbf_loops_forward(const int8_t *S_A, const int8_t *S_B,
                       const double *U_A, const double *V_A,
                       const double *U_B, const double *V_B,
                       int d_out, int d_in, int k, int l,
                       const double *X, int T, double *W, double *Y)
{
    int rc = mdbf_loops_reconstruct(S_A, S_B, U_A, V_A, U_B, V_B, d_out, d_in, k, l, W);
    if (rc) return rc;
    for (int n = 0; n < d_out; ++n)
        for (int tau = 0; tau < T; ++tau) {
            double y = 0.0;
            for (int i = 0; i < d_in; ++i) y += W[(size_t)n * d_in + i] * X[(size_t)i * T + tau];
            Y[(size_t)n * T + tau] = y;
        }
    return 0;
}

/* Bit packing by definition: word c/32 of a row, bit c%32 (LSB = 0), set <=> -1. */
int mdbf_loops_pack(const int8_t *S, int64_t rows, int64_t cols, uint32_t *out)
{
    int64_t nw = (cols + 31) / 32;
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t w = 0; w < nw; ++w) out[r * nw + w] = 0u;
        for (int64_t c = 0; c < cols; ++c) {
            int8_t s = S[r * cols + c];
            if (s != 1 && s != -1) return -1;
            if (s == -1) out[r * nw + c / 32] |= (uint32_t)1u << (unsigned)(c % 32);
        }
    }
    return 0;
}
