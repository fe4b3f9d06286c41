/*
 * CPU oracle for the operator-split linear layer.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the CUDA path is checked against.
 * It shares no code with the CUDA path and must never be called from the product:
 * only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it follows.  The paper's Section 3.3 ("Operator Splitting") gives the method
 * in three steps: (1) partition the operator and the matching dimension of its input
 * into `slice granularity` slices, (2) compute the slices one after another, (3) sum
 * the partial results.  Everything is fp64 arithmetic on values that were first
 * rounded to bfloat16 (the bit patterns the GPU receives).
 *
 * Notation: X [M,K] tokens x in_features, W [N,K] out_features x in_features
 * (row-major, Y = X W^T), b [N], dY/Y [M,N].  k = number of slices.
 *   OUT split: the N rows of W are cut into k row ranges R_s (outputs concatenate,
 *              dX is the sum over slices).
 *   RED split: the K columns of W and of X are cut into k column ranges C_s (this is
 *              the split Section 3.3 describes: the input is cut along its last dimension and the
 *              slice products are added up).
 * The split routines are written as literal loops over slices on sub-matrix views;
 * they do not call the unsplit routines, so "split == unsplit" is a test, not an
 * identity by construction.
 *
 * Readings where the paper is silent: slice length = ceil(D/k) rounded up to a
 * multiple of 8 elements; slices summed in ascending order; bias added once; the
 * activation applied once after the full sum; backward derived by differentiation.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_BAD_SPLIT 1
#define ORC_BAD_ARG 2

#define ACT_NONE 0
#define ACT_GELU_TANH 1
#define ACT_GELU_ERF 2

#define SPLIT_OUT 0
#define SPLIT_RED 1

/* ---------------------------------------------------------------- bf16 <-> fp64 */

/* Exact widening: a bf16 value is the top 16 bits of an fp32 value. */
void orc_bf16_to_f64(const uint16_t *in, double *out, size_t n)
{
    for (size_t i = 0; i < n; ++i) {
        uint32_t u = (uint32_t)in[i] << 16;
        float f;
        memcpy(&f, &u, 4);
        out[i] = (double)f;
    }
}

/* fp32 -> bf16, round to nearest, ties to even; NaN stays NaN, Inf stays Inf. */
void orc_f32_to_bf16(const float *in, uint16_t *out, size_t n)
{
    for (size_t i = 0; i < n; ++i) {
        uint32_t u;
        memcpy(&u, &in[i], 4);
        if ((u & 0x7F800000u) == 0x7F800000u) { /* Inf or NaN: truncate, keep NaN a NaN */
            uint16_t h = (uint16_t)(u >> 16);
            if ((u & 0x007FFFFFu) != 0 && (h & 0x007Fu) == 0) h |= 0x0040u;
            out[i] = h;
            continue;
        }
        uint32_t lower = u & 0xFFFFu;
        uint32_t upper = u >> 16;
        if (lower > 0x8000u || (lower == 0x8000u && (upper & 1u))) upper += 1u;
        out[i] = (uint16_t)upper;
    }
}

/* ---------------------------------------------------------------- fp8 (e4m3) -> fp64 */

/* Exact widening of the 8-bit format with 1 sign, 4 exponent (bias 7) and 3 mantissa bits, the
 * variant without infinities: exponent 15 with mantissa 7 is NaN, every other code is finite
 * (largest 448); exponent 0 holds the subnormals m/8 * 2^-6. */
void orc_e4m3_to_f64(const uint8_t *in, double *out, size_t n)
{
    for (size_t i = 0; i < n; ++i) {
        const int sign = in[i] >> 7, e = (in[i] >> 3) & 15, m = in[i] & 7;
        double v;
        if (e == 15 && m == 7) v = NAN;
        else if (e == 0) v = ldexp((double)m / 8.0, -6);
        else v = ldexp(1.0 + (double)m / 8.0, e - 7);
        out[i] = sign ? -v : v;
    }
}

/* ---------------------------------------------------------------- GeLU */

static const double kSqrt2OverPi = 0.79788456080286535587989211986876;
static const double kInvSqrt2 = 0.70710678118654752440084436210485;
static const double kInvSqrt2Pi = 0.39894228040143267793994605993438;

double orc_gelu(double x, int act)
{
    if (act == ACT_GELU_TANH) {
        double u = kSqrt2OverPi * (x + 0.044715 * x * x * x);
        return 0.5 * x * (1.0 + tanh(u));
    }
    if (act == ACT_GELU_ERF) return 0.5 * x * (1.0 + erf(x * kInvSqrt2));
    return x;
}

double orc_gelu_grad(double x, int act)
{
    if (act == ACT_GELU_TANH) {
        double u = kSqrt2OverPi * (x + 0.044715 * x * x * x);
        double t = tanh(u);
        double du = kSqrt2OverPi * (1.0 + 3.0 * 0.044715 * x * x);
        return 0.5 * (1.0 + t) + 0.5 * x * (1.0 - t * t) * du;
    }
    if (act == ACT_GELU_ERF) {
        double Phi = 0.5 * (1.0 + erf(x * kInvSqrt2));
        double phi = kInvSqrt2Pi * exp(-0.5 * x * x);
        return Phi + x * phi;
    }
    return 1.0;
}

/* ---------------------------------------------------------------- slice table */

/* Slice s of a dimension of extent D cut into k slices: [begin, end).
 * L = ceil(D/k) rounded up to a multiple of 8; every slice must be non-empty. */
int orc_slice_range(long D, int k, int s, long *begin, long *end)
{
    if (k <= 0) k = 1; /* the paper plots granularity 0 as "no splitting" */
    if (D <= 0 || s < 0 || s >= k) return ORC_BAD_ARG;
    long L = (D + k - 1) / k;
    L = (L + 7) / 8 * 8;
    if ((long)(k - 1) * L >= D) return ORC_BAD_SPLIT;
    long b = (long)s * L;
    long e = b + L;
    if (e > D) e = D;
    *begin = b;
    *end = e;
    return ORC_OK;
}

/* ---------------------------------------------------------------- plain matrix products on views
 * Every matrix is a row-major view: pointer + leading dimension.  The three products
 * are the textbook definitions; OpenMP runs rows in parallel, nothing is blocked. */

/* C[m,n] (+)= sum_j A[m,j] * B[n,j]      A [M,J], B [N,J], C [M,N] */
static void mm_nt(const double *A, long lda, const double *B, long ldb, double *C, long ldc,
                  long M, long N, long J, int accumulate)
{
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        for (long n = 0; n < N; ++n) {
            const double *a = A + m * lda;
            const double *b = B + n * ldb;
            double acc = 0.0;
#pragma omp simd reduction(+ : acc)
            for (long j = 0; j < J; ++j) acc += a[j] * b[j];
            if (accumulate) C[m * ldc + n] += acc;
            else C[m * ldc + n] = acc;
        }
    }
}

/* C[m,j] (+)= sum_n A[m,n] * B[n,j]      A [M,N], B [N,J], C [M,J] */
static void mm_nn(const double *A, long lda, const double *B, long ldb, double *C, long ldc,
                  long M, long N, long J, int accumulate)
{
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        double *c = C + m * ldc;
        if (!accumulate)
            for (long j = 0; j < J; ++j) c[j] = 0.0;
        for (long n = 0; n < N; ++n) {
            double a = A[m * lda + n];
            const double *b = B + n * ldb;
#pragma omp simd
            for (long j = 0; j < J; ++j) c[j] += a * b[j];
        }
    }
}

/* C[n,j] (+)= sum_m A[m,n] * B[m,j]      A [M,N], B [M,J], C [N,J] */
static void mm_tn(const double *A, long lda, const double *B, long ldb, double *C, long ldc,
                  long M, long N, long J, int accumulate)
{
#pragma omp parallel for schedule(static)
    for (long n = 0; n < N; ++n) {
        double *c = C + n * ldc;
        if (!accumulate)
            for (long j = 0; j < J; ++j) c[j] = 0.0;
        for (long m = 0; m < M; ++m) {
            double a = A[m * lda + n];
            const double *b = B + m * ldb;
#pragma omp simd
            for (long j = 0; j < J; ++j) c[j] += a * b[j];
        }
    }
}

/* ---------------------------------------------------------------- unsplit linear */

/* Z = X W^T + b, Y = act(Z).  Z (pre-activation) may be NULL; b may be NULL. */
int orc_linear_fwd(const double *X, const double *W, const double *b, long M, long N, long K,
                   int act, double *Z, double *Y)
{
    if (!X || !W || !Y || M <= 0 || N <= 0 || K <= 0) return ORC_BAD_ARG;
    mm_nt(X, K, W, K, Y, N, M, N, K, 0);
    for (long m = 0; m < M; ++m)
        for (long n = 0; n < N; ++n) {
            double z = Y[m * N + n] + (b ? b[n] : 0.0);
            if (Z) Z[m * N + n] = z;
            Y[m * N + n] = orc_gelu(z, act);
        }
    return ORC_OK;
}

/* G = dY (.) act'(Z);  dX = G W;  dW = G^T X;  db = column sums of G.
 * Z is the pre-activation from the forward (ignored when act is none). Outputs may be NULL. */
int orc_linear_bwd(const double *dY, const double *X, const double *W, const double *Z,
                   long M, long N, long K, int act, double *dX, double *dW, double *db)
{
    if (!dY || !X || !W || M <= 0 || N <= 0 || K <= 0) return ORC_BAD_ARG;
    if (act != ACT_NONE && !Z) return ORC_BAD_ARG;
    double *G = (double *)malloc(sizeof(double) * (size_t)M * (size_t)N);
    if (!G) return ORC_BAD_ARG;
    for (long i = 0; i < M * N; ++i) G[i] = dY[i] * (act == ACT_NONE ? 1.0 : orc_gelu_grad(Z[i], act));
    if (dX) mm_nn(G, N, W, K, dX, K, M, N, K, 0);
    if (dW) mm_tn(G, N, X, K, dW, K, M, N, K, 0);
    if (db)
        for (long n = 0; n < N; ++n) {
            double s = 0.0;
            for (long m = 0; m < M; ++m) s += G[m * N + n];
            db[n] = s;
        }
    free(G);
    return ORC_OK;
}

/* ---------------------------------------------------------------- split linear: loops over slices */

/* Forward, k slices processed one after another (Section 3.3, steps 1-3).
 *  OUT: slice s owns rows R_s of W; it produces columns R_s of Z and Y (concatenation).
 *  RED: slice s owns columns C_s of X and of W; partial products are summed in
 *       ascending s; bias and activation are applied once after the last slice. */
int orc_split_linear_fwd(const double *X, const double *W, const double *b, long M, long N, long K,
                         int k, int split_dim, int act, double *Z, double *Y)
{
    if (!X || !W || !Y || M <= 0 || N <= 0 || K <= 0) return ORC_BAD_ARG;
    if (k <= 0) k = 1;
    long lo, hi;
    if (split_dim == SPLIT_OUT) {
        for (int s = 0; s < k; ++s) {
            int rc = orc_slice_range(N, k, s, &lo, &hi);
            if (rc) return rc;
            /* W_s = W[lo:hi, :]  ->  Y[:, lo:hi] */
            mm_nt(X, K, W + lo * K, K, Y + lo, N, M, hi - lo, K, 0);
            for (long m = 0; m < M; ++m)
                for (long n = lo; n < hi; ++n) {
                    double z = Y[m * N + n] + (b ? b[n] : 0.0);
                    if (Z) Z[m * N + n] = z;
                    Y[m * N + n] = orc_gelu(z, act);
                }
        }
        return ORC_OK;
    }
    if (split_dim == SPLIT_RED) {
        for (int s = 0; s < k; ++s) {
            int rc = orc_slice_range(K, k, s, &lo, &hi);
            if (rc) return rc;
            /* P_s = X[:, lo:hi] W[:, lo:hi]^T, summed into Y */
            mm_nt(X + lo, K, W + lo, K, Y, N, M, N, hi - lo, s > 0);
        }
        for (long m = 0; m < M; ++m)
            for (long n = 0; n < N; ++n) {
                double z = Y[m * N + n] + (b ? b[n] : 0.0);
                if (Z) Z[m * N + n] = z;
                Y[m * N + n] = orc_gelu(z, act);
            }
        return ORC_OK;
    }
    return ORC_BAD_ARG;
}

/* Backward, slice by slice.
 *  OUT: G_s = G[:, R_s];  dW[R_s,:] = G_s^T X;  db[R_s] = colsum G_s;  dX = sum_s G_s W[R_s,:].
 *  RED: dX[:, C_s] = G W[:, C_s];  dW[:, C_s] = G^T X[:, C_s];  db = colsum G. */
int orc_split_linear_bwd(const double *dY, const double *X, const double *W, const double *Z,
                         long M, long N, long K, int k, int split_dim, int act,
                         double *dX, double *dW, double *db)
{
    if (!dY || !X || !W || M <= 0 || N <= 0 || K <= 0) return ORC_BAD_ARG;
    if (act != ACT_NONE && !Z) return ORC_BAD_ARG;
    if (k <= 0) k = 1;
    double *G = (double *)malloc(sizeof(double) * (size_t)M * (size_t)N);
    if (!G) return ORC_BAD_ARG;
    long lo, hi;
    int rc = ORC_OK;
    if (split_dim == SPLIT_OUT) {
        for (int s = 0; s < k && !rc; ++s) {
            rc = orc_slice_range(N, k, s, &lo, &hi);
            if (rc) break;
            for (long m = 0; m < M; ++m)
                for (long n = lo; n < hi; ++n)
                    G[m * N + n] = dY[m * N + n] * (act == ACT_NONE ? 1.0 : orc_gelu_grad(Z[m * N + n], act));
            if (dX) mm_nn(G + lo, N, W + lo * K, K, dX, K, M, hi - lo, K, s > 0);
            if (dW) mm_tn(G + lo, N, X, K, dW + lo * K, K, M, hi - lo, K, 0);
            if (db)
                for (long n = lo; n < hi; ++n) {
                    double acc = 0.0;
                    for (long m = 0; m < M; ++m) acc += G[m * N + n];
                    db[n] = acc;
                }
        }
    } else if (split_dim == SPLIT_RED) {
        for (long i = 0; i < M * N; ++i) G[i] = dY[i] * (act == ACT_NONE ? 1.0 : orc_gelu_grad(Z[i], act));
        for (int s = 0; s < k && !rc; ++s) {
            rc = orc_slice_range(K, k, s, &lo, &hi);
            if (rc) break;
            if (dX) mm_nn(G, N, W + lo, K, dX + lo, K, M, N, hi - lo, 0);
            if (dW) mm_tn(G, N, X + lo, K, dW + lo, K, M, N, hi - lo, 0);
        }
        if (db && !rc)
            for (long n = 0; n < N; ++n) {
                double acc = 0.0;
                for (long m = 0; m < M; ++m) acc += G[m * N + n];
                db[n] = acc;
            }
    } else {
        rc = ORC_BAD_ARG;
    }
    free(G);
    return rc;
}

/* ---------------------------------------------------------------- MLP block: Linear -> GeLU -> Linear
 * X [M,H], W1 [F,H], b1 [F], W2 [H,F], b2 [H]; Z1 = X W1^T + b1, A = gelu(Z1), Y = A W2^T + b2.
 * Nothing is rounded between the two layers (the oracle's inputs are rounded, not its
 * intermediates). */

int orc_mlp_fwd(const double *X, const double *W1, const double *b1, const double *W2, const double *b2,
                long M, long H, long F, int act, double *Z1, double *Y)
{
    if (!X || !W1 || !W2 || !Y || M <= 0 || H <= 0 || F <= 0) return ORC_BAD_ARG;
    double *A = (double *)malloc(sizeof(double) * (size_t)M * (size_t)F);
    if (!A) return ORC_BAD_ARG;
    int rc = orc_linear_fwd(X, W1, b1, M, F, H, act, Z1, A);
    if (!rc) rc = orc_linear_fwd(A, W2, b2, M, H, F, ACT_NONE, NULL, Y);
    free(A);
    return rc;
}

/* dA = dY W2;  dZ1 = dA (.) act'(Z1);  dW2 = dY^T A;  db2 = colsum dY;
 * dW1 = dZ1^T X;  db1 = colsum dZ1;  dX = dZ1 W1.   Z1 is recomputed here from X, W1, b1. */
int orc_mlp_bwd(const double *dY, const double *X, const double *W1, const double *b1, const double *W2,
                long M, long H, long F, int act,
                double *dX, double *dW1, double *db1, double *dW2, double *db2)
{
    if (!dY || !X || !W1 || !W2 || M <= 0 || H <= 0 || F <= 0) return ORC_BAD_ARG;
    size_t mf = (size_t)M * (size_t)F;
    double *Z1 = (double *)malloc(sizeof(double) * mf);
    double *A = (double *)malloc(sizeof(double) * mf);
    double *dA = (double *)malloc(sizeof(double) * mf);
    if (!Z1 || !A || !dA) { free(Z1); free(A); free(dA); return ORC_BAD_ARG; }
    int rc = orc_linear_fwd(X, W1, b1, M, F, H, act, Z1, A);
    if (!rc) {
        /* second layer backward (no activation): input A, weight W2 [H,F] */
        rc = orc_linear_bwd(dY, A, W2, NULL, M, H, F, ACT_NONE, dA, dW2, db2);
    }
    if (!rc) {
        /* first layer backward: upstream dA, activation derivative at Z1 */
        rc = orc_linear_bwd(dA, X, W1, Z1, M, F, H, act, dX, dW1, db1);
    }
    free(Z1); free(A); free(dA);
    return rc;
}

/* Split along the ffn dimension F into k slices F_s (first layer OUT-split, second layer
 * RED-split):  Y = sum_s gelu(X W1[F_s,:]^T + b1[F_s]) W2[:,F_s]^T + b2, one slice at a time;
 * only slice-sized intermediates (A_s, Z1_s) exist. */
int orc_split_mlp_fwd(const double *X, const double *W1, const double *b1, const double *W2, const double *b2,
                      long M, long H, long F, int k, int act, double *Y)
{
    if (!X || !W1 || !W2 || !Y || M <= 0 || H <= 0 || F <= 0) return ORC_BAD_ARG;
    if (k <= 0) k = 1;
    long lo, hi;
    int rc = orc_slice_range(F, k, 0, &lo, &hi);
    if (rc) return rc;
    long L = hi - lo;
    double *As = (double *)malloc(sizeof(double) * (size_t)M * (size_t)L);
    if (!As) return ORC_BAD_ARG;
    for (int s = 0; s < k; ++s) {
        rc = orc_slice_range(F, k, s, &lo, &hi);
        if (rc) break;
        long Ls = hi - lo;
        mm_nt(X, H, W1 + lo * H, H, As, Ls, M, Ls, H, 0);
        for (long m = 0; m < M; ++m)
            for (long f = 0; f < Ls; ++f)
                As[m * Ls + f] = orc_gelu(As[m * Ls + f] + (b1 ? b1[lo + f] : 0.0), act);
        mm_nt(As, Ls, W2 + lo, F, Y, H, M, H, Ls, s > 0);
    }
    if (!rc)
        for (long m = 0; m < M; ++m)
            for (long h = 0; h < H; ++h) Y[m * H + h] += (b2 ? b2[h] : 0.0);
    free(As);
    return rc;
}

/* Backward of the split MLP, slice by slice (Z1_s recomputed per slice):
 *  dA_s = dY W2[:,F_s];  dZ_s = dA_s (.) act'(Z1_s);  dW2[:,F_s] = dY^T A_s;
 *  dW1[F_s,:] = dZ_s^T X;  db1[F_s] = colsum dZ_s;  dX = sum_s dZ_s W1[F_s,:];  db2 = colsum dY. */
int orc_split_mlp_bwd(const double *dY, const double *X, const double *W1, const double *b1, const double *W2,
                      long M, long H, long F, int k, int act,
                      double *dX, double *dW1, double *db1, double *dW2, double *db2)
{
    if (!dY || !X || !W1 || !W2 || M <= 0 || H <= 0 || F <= 0) return ORC_BAD_ARG;
    if (k <= 0) k = 1;
    long lo, hi;
    int rc = orc_slice_range(F, k, 0, &lo, &hi);
    if (rc) return rc;
    long L = hi - lo;
    size_t ml = (size_t)M * (size_t)L;
    double *Zs = (double *)malloc(sizeof(double) * ml);
    double *As = (double *)malloc(sizeof(double) * ml);
    double *dZs = (double *)malloc(sizeof(double) * ml);
    if (!Zs || !As || !dZs) { free(Zs); free(As); free(dZs); return ORC_BAD_ARG; }
    for (int s = 0; s < k; ++s) {
        rc = orc_slice_range(F, k, s, &lo, &hi);
        if (rc) break;
        long Ls = hi - lo;
        mm_nt(X, H, W1 + lo * H, H, Zs, Ls, M, Ls, H, 0);
        for (long m = 0; m < M; ++m)
            for (long f = 0; f < Ls; ++f) {
                double z = Zs[m * Ls + f] + (b1 ? b1[lo + f] : 0.0);
                Zs[m * Ls + f] = z;
                As[m * Ls + f] = orc_gelu(z, act);
            }
        /* dA_s [M,Ls] = dY [M,H] * W2[:, lo:hi] [H,Ls] */
        mm_nn(dY, H, W2 + lo, F, dZs, Ls, M, H, Ls, 0);
        for (long i = 0; i < M * Ls; ++i) dZs[i] *= orc_gelu_grad(Zs[i], act);
        /* dW2[:, lo:hi] [H,Ls] = dY^T [H,M] * A_s [M,Ls] */
        if (dW2) mm_tn(dY, H, As, Ls, dW2 + lo, F, M, H, Ls, 0);
        /* dW1[lo:hi, :] [Ls,H] = dZ_s^T [Ls,M] * X [M,H] */
        if (dW1) mm_tn(dZs, Ls, X, H, dW1 + lo * H, H, M, Ls, H, 0);
        if (db1)
            for (long f = 0; f < Ls; ++f) {
                double acc = 0.0;
                for (long m = 0; m < M; ++m) acc += dZs[m * Ls + f];
                db1[lo + f] = acc;
            }
        /* dX [M,H] += dZ_s [M,Ls] * W1[lo:hi, :] [Ls,H] */
        if (dX) mm_nn(dZs, Ls, W1 + lo * H, H, dX, H, M, Ls, H, s > 0);
    }
    if (db2 && !rc)
        for (long h = 0; h < H; ++h) {
            double acc = 0.0;
            for (long m = 0; m < M; ++m) acc += dY[m * H + h];
            db2[h] = acc;
        }
    free(Zs); free(As); free(dZs);
    return rc;
}

int orc_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
