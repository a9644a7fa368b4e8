/*
 * CPU oracle for the GEMM hot path  C = alpha * op(A) * op(B) + beta * C.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may link or call this file; it shares
 * no code, header, table or helper with the CUDA library.  It is deliberately plain and slow.
 *
 * Two layers:
 *   L0  the definition (Section II-A: C = C + A B with A m x k, B k x n, C m x n), written as
 *       one dot product per entry summed in increasing k, with the alpha/beta form of the
 *       micro-kernel of Fig. 3 folded in as  alpha*acc + beta*C0.
 *   L1  the paper's method: the five loops jc/pc/ic/jr/ir of Fig. 1 around Pack-B, Pack-A and a
 *       micro-kernel that performs kc rank-1 updates on an mr x nr block (Fig. 3 / Fig. 4),
 *       packed panels Ac[kc][mr], Bc[kc][nr] zero-padded to whole mr / nr (Section III-A).
 *
 * Storage convention: BLAS column-major, element (i,j) of X is X[i + j*ldx].
 * Every function is pinned by tests that do not come from this file (closed forms, hand-worked
 * examples, brute force, exact integer cases); no function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { OR_F32 = 0, OR_F16 = 1, OR_BF16 = 2 };
enum { ACC_F32 = 0, ACC_F32FMA = 1, ACC_F64 = 2, ACC_F16 = 3 };

/* ---------------------------------------------------------------- element decoding */

/* IEEE binary16 -> double, from the format's definition: 1 sign, 5 exponent (bias 15), 10 fraction bits */
double oracle_decode_f16(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1F;
    int f = h & 0x3FF;
    double v;
    if (e == 0)        v = ldexp((double)f, -24);                 /* subnormal: f * 2^-10 * 2^-14 */
    else if (e == 31)  v = f ? NAN : INFINITY;
    else               v = ldexp((double)(f | 0x400), e - 25);    /* (1 + f/1024) * 2^(e-15) */
    return sign ? -v : v;
}

/* bfloat16 -> double: the 16 bits are the upper half of a binary32 (1 sign, 8 exponent bias 127, 7 fraction) */
double oracle_decode_bf16(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 7) & 0xFF;
    int f = h & 0x7F;
    double v;
    if (e == 0)        v = ldexp((double)f, -133);                /* f * 2^-7 * 2^-126 */
    else if (e == 255) v = f ? NAN : INFINITY;
    else               v = ldexp((double)(f | 0x80), e - 134);    /* (1 + f/128) * 2^(e-127) */
    return sign ? -v : v;
}

/*
 * Nearest IEEE binary16 number to x, ties to even, returned as a double (from the format's definition: 11
 * significant bits, exponents -14 .. 15, subnormals in steps of 2^-24, overflow to infinity from 65520 on).
 */
double oracle_round_f16(double x) {
    if (isnan(x) || isinf(x) || x == 0.0) return x;
    double ax = fabs(x);
    int e;
    frexp(ax, &e);                    /* ax = f * 2^e, 0.5 <= f < 1: the leading bit has weight 2^(e-1) */
    int lsb = e - 11;                 /* weight of the last of 11 significant bits */
    if (lsb < -24) lsb = -24;         /* subnormal range: fixed spacing 2^-24 */
    double q = ldexp(ax, -lsb);       /* in units of the last place: exact scaling */
    double r = nearbyint(q);          /* default rounding mode: to nearest, ties to even */
    double v = ldexp(r, lsb);
    if (v >= 65520.0) v = INFINITY;   /* 65504 is the largest finite value; halfway to 2^16 rounds up */
    return x < 0 ? -v : v;
}

static inline double elem(const void* X, int dtype, int64_t idx) {
    if (dtype == OR_F32) return (double)((const float*)X)[idx];
    if (dtype == OR_F16) return oracle_decode_f16(((const uint16_t*)X)[idx]);
    return oracle_decode_bf16(((const uint16_t*)X)[idx]);
}

/* op(A)(i,p): A stored m x k when not transposed, k x m when transposed */
static inline double opA(const void* A, int dtype, int ta, int64_t lda, int64_t i, int64_t p) {
    return elem(A, dtype, ta ? p + i * lda : i + p * lda);
}
/* op(B)(p,j): B stored k x n when not transposed, n x k when transposed */
static inline double opB(const void* B, int dtype, int tb, int64_t ldb, int64_t p, int64_t j) {
    return elem(B, dtype, tb ? j + p * ldb : p + j * ldb);
}

/* ---------------------------------------------------------------- L0: the definition */

/*
 * Brute force.  acc in {ACC_F32, ACC_F32FMA}: result written to C32 (C64 ignored);
 * ACC_F64: result written to C64 and, if C32 != NULL, rounded once to float there;
 * ACC_F16: the dot product is accumulated in binary16, then alpha*sum + beta*C0 is formed in double and written like ACC_F64.
 * C0 (fp32, ldc0) is read only when beta != 0.
 */
int oracle_gemm_l0(int dtype, int acc, int ta, int tb, int64_t m, int64_t n, int64_t k,
                   double alpha, const void* A, int64_t lda, const void* B, int64_t ldb,
                   double beta, const float* C0, int64_t ldc0,
                   double* C64, float* C32, int64_t ldc) {
    if (m < 0 || n < 0 || k < 0) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < n; ++j) {
        for (int64_t i = 0; i < m; ++i) {
            if (acc == ACC_F64 || acc == ACC_F16) {
                double s = 0.0;
                if (acc == ACC_F64) {
                    for (int64_t p = 0; p < k; ++p)
                        s += opA(A, dtype, ta, lda, i, p) * opB(B, dtype, tb, ldb, p, j);
                } else {
                    /* the paper's f16 arithmetic (Section III-D): the running sum is a binary16 number, updated by one
                     * fused multiply-add per k (the product of two binary16 numbers and its sum with a third are exact
                     * in double; one rounding to binary16) */
                    for (int64_t p = 0; p < k; ++p)
                        s = oracle_round_f16(s + opA(A, dtype, ta, lda, i, p) * opB(B, dtype, tb, ldb, p, j));
                }
                double r = alpha * s;
                if (beta != 0.0) r += beta * (double)C0[i + j * ldc0];
                if (C64) C64[i + j * ldc] = r;
                if (C32) C32[i + j * ldc] = (float)r;
            } else {
                float s = 0.0f;
                const float al = (float)alpha, be = (float)beta;
                for (int64_t p = 0; p < k; ++p) {
                    float a = (float)opA(A, dtype, ta, lda, i, p);
                    float b = (float)opB(B, dtype, tb, ldb, p, j);
                    if (acc == ACC_F32FMA) s = fmaf(a, b, s);
                    else { float t = a * b; s = s + t; }
                }
                float c0 = (beta != 0.0) ? be * C0[i + j * ldc0] : 0.0f;
                float r;
                if (acc == ACC_F32FMA) r = fmaf(al, s, c0);
                else { float t = al * s; r = c0 + t; }
                C32[i + j * ldc] = r;
            }
        }
    }
    return 0;
}

/* fp64 value of selected entries (is[t], js[t]) of alpha*op(A)op(B) + beta*C0: for shapes too large for L0 */
int oracle_gemm_samples_f64(int dtype, int ta, int tb, int64_t k,
                            double alpha, const void* A, int64_t lda, const void* B, int64_t ldb,
                            double beta, const float* C0, int64_t ldc0,
                            int64_t nsamples, const int64_t* is, const int64_t* js, double* out) {
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t t = 0; t < nsamples; ++t) {
        double s = 0.0;
        for (int64_t p = 0; p < k; ++p)
            s += opA(A, dtype, ta, lda, is[t], p) * opB(B, dtype, tb, ldb, p, js[t]);
        double r = alpha * s;
        if (beta != 0.0) r += beta * (double)C0[is[t] + js[t] * ldc0];
        out[t] = r;
    }
    return 0;
}

/*
 * Randomised whole-matrix check (Freivalds): for a probe vector x (length n) returns
 *   resid = C x - ( alpha * op(A) (op(B) x) + beta * C0 x )      (length m, fp64)
 *   scale = |alpha| * |op(A)| (|op(B)| |x|) + |beta| * |C0| |x|  (length m): the magnitude to judge resid against.
 * C is the fp32 result under test.  Cost O(mk + kn + mn).
 */
int oracle_freivalds(int dtype, int ta, int tb, int64_t m, int64_t n, int64_t k,
                     double alpha, const void* A, int64_t lda, const void* B, int64_t ldb,
                     double beta, const float* C0, int64_t ldc0, const float* C, int64_t ldc,
                     const double* x, double* resid, double* scale) {
    double* bx = (double*)malloc(sizeof(double) * (size_t)(k > 0 ? k : 1));
    double* bxa = (double*)malloc(sizeof(double) * (size_t)(k > 0 ? k : 1));
    if (!bx || !bxa) { free(bx); free(bxa); return -2; }
#pragma omp parallel for schedule(static)
    for (int64_t p = 0; p < k; ++p) {
        double s = 0.0, sa = 0.0;
        for (int64_t j = 0; j < n; ++j) {
            double b = opB(B, dtype, tb, ldb, p, j);
            s += b * x[j];
            sa += fabs(b) * fabs(x[j]);
        }
        bx[p] = s; bxa[p] = sa;
    }
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i) {
        double s = 0.0, sa = 0.0, cx = 0.0, c0x = 0.0, c0a = 0.0;
        for (int64_t p = 0; p < k; ++p) {
            double a = opA(A, dtype, ta, lda, i, p);
            s += a * bx[p];
            sa += fabs(a) * bxa[p];
        }
        for (int64_t j = 0; j < n; ++j) cx += (double)C[i + j * ldc] * x[j];
        if (beta != 0.0)
            for (int64_t j = 0; j < n; ++j) {
                double c0 = (double)C0[i + j * ldc0];
                c0x += c0 * x[j];
                c0a += fabs(c0) * fabs(x[j]);
            }
        resid[i] = cx - (alpha * s + beta * c0x);
        scale[i] = fabs(alpha) * sa + fabs(beta) * c0a;
    }
    free(bx); free(bxa);
    return 0;
}

/* ---------------------------------------------------------------- L1: packed, blocked GEMM */

#define T float
#define SUFFIX f32
#include "gemm_l1_body.inc"
#undef T
#undef SUFFIX

#define T double
#define SUFFIX f64
#include "gemm_l1_body.inc"
#undef T
#undef SUFFIX

/*
 * acc == ACC_F32: C is float* (in: C0, out: result), arithmetic in float (mul then add, no contraction).
 * acc == ACC_F64: C is double* (in: C0 widened by the caller, out: result), arithmetic in double.
 * paper_scaling != 0 places the scalars where Fig. 3 has them (alpha on the packed B panel, beta on the tile of C
 * the sums start from); otherwise the block contribution is accumulated from zero and folded in as
 * alpha*acc + beta*C.
 */
int oracle_gemm_l1(int dtype, int acc, int ta, int tb, int64_t m, int64_t n, int64_t k,
                   double alpha, const void* A, int64_t lda, const void* B, int64_t ldb,
                   double beta, void* C, int64_t ldc,
                   int mr, int nr, int mc, int kc, int nc, int paper_scaling) {
    if (m < 0 || n < 0 || k < 0 || mr <= 0 || nr <= 0 || mc <= 0 || kc <= 0 || nc <= 0) return -1;
    if (mr > 64 || nr > 64) return -1;
    if (acc == ACC_F32)
        return gemm_l1_f32(dtype, ta, tb, m, n, k, (float)alpha, A, lda, B, ldb, (float)beta,
                           (float*)C, ldc, mr, nr, mc, kc, nc, paper_scaling);
    if (acc == ACC_F64)
        return gemm_l1_f64(dtype, ta, tb, m, n, k, alpha, A, lda, B, ldb, beta,
                           (double*)C, ldc, mr, nr, mc, kc, nc, paper_scaling);
    return -1;
}

/* the packing routines on their own, for the layout tests (float panels) */
int oracle_pack_A_f32(int dtype, int ta, const void* A, int64_t lda, int64_t ic, int64_t pc,
                      int64_t mcb, int64_t kcb, int mr, float* Ac) {
    pack_A_f32(dtype, ta, A, lda, ic, pc, mcb, kcb, mr, Ac);
    return 0;
}
int oracle_pack_B_f32(int dtype, int tb, const void* B, int64_t ldb, int64_t pc, int64_t jc,
                      int64_t kcb, int64_t ncb, int nr, float* Bc) {
    pack_B_f32(dtype, tb, B, ldb, pc, jc, kcb, ncb, nr, Bc, 0, 1.0f);
    return 0;
}

/* one full tile through the micro-kernel, with the argument list of Fig. 3 (C is the contiguous [NR][MR]
 * block), float.  In the paper's placement of the scalars the B panel is scaled the way Pack-B scales it. */
int oracle_ukernel_f32(int mr, int nr, int64_t kc, float alpha, const float* Ac, const float* Bc,
                       float beta, float* C, int paper_scaling) {
    if (mr > 64 || nr > 64) return -1;
    const float* Bp = Bc;
    float* scaled = NULL;
    if (paper_scaling) {
        scaled = (float*)malloc(sizeof(float) * (size_t)(kc > 0 ? kc : 1) * (size_t)nr);
        if (!scaled) return -2;
        for (int64_t e = 0; e < kc * nr; ++e) scaled[e] = Bc[e] * alpha;
        Bp = scaled;
    }
    tile_update_f32(mr, nr, mr, nr, kc, alpha, beta, Ac, Bp, C, mr, paper_scaling);
    free(scaled);
    return 0;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
