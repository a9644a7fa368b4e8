/*
 * CPU oracle for the convolution layers that the paper lowers to GEMM with the im2row transform
 * (Section IV-C, "Rectangular Matrices": the GEMM dimensions of its Tables "resnet50" and "vgg16"
 * are m = batch*Ho*Wo output pixels, n = C_out, k = C_in*kh*kw).
 *
 * TEST INFRASTRUCTURE ONLY, like the rest of this directory: nothing on the product path links or calls it,
 * and it shares no code with the CUDA library.
 *
 * Two independent routes to the same numbers:
 *   direct   the textbook definition of a 2-D cross-correlation layer with zero padding, one fp64 sum per output
 *            entry over (r, s, c) in that order;
 *   im2row   the lowering itself: row j of the lowered matrix is the receptive field ("patch") of output pixel j,
 *            k = kh*kw*C_in entries in (r, s, c) order, zeros where the patch leaves the image.  Multiplying it
 *            by the k x C_out filter matrix (the GEMM oracle does that) must reproduce `direct` bit for bit in
 *            fp64, because both sum the same products in the same order.
 *
 * Layouts.  Activations X: NHWC, element (b, h, w, c) at ((b*H + h)*W + w)*C_in + c.  Filters: element
 * (co; r, s, c) at co + ((r*kw + s)*C_in + c)*ldw, i.e. a column-major C_out x k matrix.  Output Y: fp32/fp64,
 * element (co; b, ho, wo) at co + ((b*Ho + ho)*Wo + wo)*ldy: NHWC, which read as a column-major matrix is
 * C_out x pixels.  Ho = (H + 2*ph - kh)/sh + 1, Wo likewise.
 * Pinned by tests against a library convolution (other layout, other code), closed forms and special cases.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

double oracle_decode_f16(uint16_t h);
double oracle_decode_bf16(uint16_t h);

enum { CV_F32 = 0, CV_F16 = 1, CV_BF16 = 2 };

typedef struct {
    int64_t batch, h, w, c_in, c_out;
    int32_t kh, kw, stride_h, stride_w, pad_h, pad_w;
} conv_geom_t;

static inline double cv_elem(const void* X, int dtype, int64_t idx) {
    if (dtype == CV_F32) return (double)((const float*)X)[idx];
    if (dtype == CV_F16) return oracle_decode_f16(((const uint16_t*)X)[idx]);
    return oracle_decode_bf16(((const uint16_t*)X)[idx]);
}

static inline int64_t out_extent(int64_t in, int pad, int k, int stride) { return (in + 2 * (int64_t)pad - k) / stride + 1; }

int64_t oracle_conv_out_h(const conv_geom_t* g) { return out_extent(g->h, g->pad_h, g->kh, g->stride_h); }
int64_t oracle_conv_out_w(const conv_geom_t* g) { return out_extent(g->w, g->pad_w, g->kw, g->stride_w); }

/* one output entry by the definition, fp64 */
static double conv_entry(const conv_geom_t* g, int dtype, const void* X, const void* Wt, int64_t ldw,
                         int64_t co, int64_t b, int64_t ho, int64_t wo) {
    double acc = 0.0;
    for (int r = 0; r < g->kh; ++r) {
        const int64_t hi = ho * g->stride_h - g->pad_h + r;
        for (int s = 0; s < g->kw; ++s) {
            const int64_t wi = wo * g->stride_w - g->pad_w + s;
            const int inside = hi >= 0 && hi < g->h && wi >= 0 && wi < g->w;
            for (int64_t c = 0; c < g->c_in; ++c) {
                const double x = inside ? cv_elem(X, dtype, ((b * g->h + hi) * g->w + wi) * g->c_in + c) : 0.0;
                const int64_t p = ((int64_t)r * g->kw + s) * g->c_in + c;
                acc += x * cv_elem(Wt, dtype, co + p * ldw);
            }
        }
    }
    return acc;
}

/* Y = alpha * conv(X, W) + beta * Y0, every entry, fp64 out (ldo >= C_out).  Y0 (fp32, ldy0) is read only if beta != 0. */
int oracle_conv2d_direct(int dtype, const conv_geom_t* g, double alpha, const void* X, const void* Wt, int64_t ldw,
                         double beta, const float* Y0, int64_t ldy0, double* out, int64_t ldo) {
    const int64_t Ho = oracle_conv_out_h(g), Wo = oracle_conv_out_w(g);
    if (Ho <= 0 || Wo <= 0) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < g->batch * Ho * Wo; ++j) {
        const int64_t b = j / (Ho * Wo), ho = (j / Wo) % Ho, wo = j % Wo;
        for (int64_t co = 0; co < g->c_out; ++co) {
            const double acc = conv_entry(g, dtype, X, Wt, ldw, co, b, ho, wo);
            out[co + j * ldo] = (beta == 0.0 ? 0.0 : beta * (double)Y0[co + j * ldy0]) + alpha * acc;
        }
    }
    return 0;
}

/* the same for a list of entries (channel rows[t], pixel cols[t]) */
int oracle_conv2d_samples_f64(int dtype, const conv_geom_t* g, double alpha, const void* X, const void* Wt, int64_t ldw,
                              double beta, const float* Y0, int64_t ldy0, int64_t count, const int64_t* rows,
                              const int64_t* cols, double* out) {
    const int64_t Ho = oracle_conv_out_h(g), Wo = oracle_conv_out_w(g);
    if (Ho <= 0 || Wo <= 0) return -1;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < count; ++t) {
        const int64_t co = rows[t], j = cols[t];
        const int64_t b = j / (Ho * Wo), ho = (j / Wo) % Ho, wo = j % Wo;
        const double acc = conv_entry(g, dtype, X, Wt, ldw, co, b, ho, wo);
        out[t] = (beta == 0.0 ? 0.0 : beta * (double)Y0[co + j * ldy0]) + alpha * acc;
    }
    return 0;
}

/*
 * The im2row lowering: writes the k x pixels column-major matrix (ld >= k) whose column j is the patch of output
 * pixel j, in the element type of X (values are copied, never converted; padding positions get +0).
 */
int oracle_im2row(int dtype, const conv_geom_t* g, const void* X, void* out, int64_t ld) {
    const int64_t Ho = oracle_conv_out_h(g), Wo = oracle_conv_out_w(g);
    if (Ho <= 0 || Wo <= 0) return -1;
    const int es = dtype == CV_F32 ? 4 : 2;
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < g->batch * Ho * Wo; ++j) {
        const int64_t b = j / (Ho * Wo), ho = (j / Wo) % Ho, wo = j % Wo;
        for (int r = 0; r < g->kh; ++r)
            for (int s = 0; s < g->kw; ++s) {
                const int64_t hi = ho * g->stride_h - g->pad_h + r, wi = wo * g->stride_w - g->pad_w + s;
                const int inside = hi >= 0 && hi < g->h && wi >= 0 && wi < g->w;
                char* dst = (char*)out + (j * ld + ((int64_t)r * g->kw + s) * g->c_in) * es;
                if (inside) memcpy(dst, (const char*)X + (((b * g->h + hi) * g->w + wi) * g->c_in) * es, (size_t)g->c_in * es);
                else memset(dst, 0, (size_t)g->c_in * es);
            }
    }
    return 0;
}
