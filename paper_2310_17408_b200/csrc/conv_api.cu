// Convolution layers through the im2row lowering (Section IV-C): the front end that turns a layer into the GEMM
//     Y[C_out x pixels] = W[C_out x k] * L[k x pixels],   k = kh*kw*C_in,
// chooses how L comes to exist (fused into the GEMM kernels' operand staging, written out by im2row_kernel, or not
// needed at all), and the im2row transform itself as a kernel.
#include "internal.cuh"

namespace b200gemm {

static int g_force_lowering = 0;

static inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline int64_t rup(int64_t a, int64_t b) { return cdiv(a, b) * b; }

// ---- the transform as a copy kernel: one thread per 16-byte chunk (CHUNK = true) or per element of L.
// Column j of L is the patch of output pixel j; a (pixel, tap) pair is C_in contiguous elements of X or zeros.
template <typename T, bool CHUNK>
__global__ void __launch_bounds__(256)
im2row_kernel(const ConvIndex cv, int64_t pixels, const T* __restrict__ X, T* __restrict__ out, int64_t ld) {
    constexpr int PER = CHUNK ? (int)(16 / sizeof(T)) : 1;          // elements moved by one thread
    const int64_t per_tap = cv.c_in / PER;                          // threads per (pixel, tap)
    const int64_t taps = (int64_t)cv.kh * cv.kw;
    const int64_t total = pixels * taps * per_tap;
    const int hw = cv.ho * cv.wo;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t j = idx / (taps * per_tap);
        const int64_t within = idx - j * (taps * per_tap);
        const int tap = (int)(within / per_tap);
        const int64_t c = (within - (int64_t)tap * per_tap) * PER;
        const int fr = tap / cv.kw, fs = tap - fr * cv.kw;
        const int b = (int)(j / hw), rem = (int)(j - (int64_t)b * hw);
        const int oh = rem / cv.wo, ow = rem - oh * cv.wo;
        const int hi = oh * cv.sh - cv.ph + fr, wi = ow * cv.sw - cv.pw + fs;
        const bool inside = (unsigned)hi < (unsigned)cv.h && (unsigned)wi < (unsigned)cv.w;
        const int64_t src = (((int64_t)b * cv.h + hi) * cv.w + wi) * cv.c_in + c;
        const int64_t dst = j * ld + (int64_t)tap * cv.c_in + c;
        if (CHUNK) {
            const uint4 v = inside ? __ldg(reinterpret_cast<const uint4*>(X + src)) : make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4*>(out + dst) = v;
        } else {
            out[dst] = inside ? X[src] : T(0);
        }
    }
}

template <typename T>
static cudaError_t launch_im2row_t(const ConvIndex& cv, int64_t pixels, const void* X, void* out, int64_t ld, cudaStream_t s) {
    const int es = (int)sizeof(T);
    const bool chunk = (cv.c_in * es) % 16 == 0 && (ld * es) % 16 == 0 && (reinterpret_cast<uintptr_t>(X) & 15) == 0 &&
                       (reinterpret_cast<uintptr_t>(out) & 15) == 0;
    const int64_t per = chunk ? 16 / es : 1;
    const int64_t total = pixels * cv.kh * cv.kw * (cv.c_in / per);
    if (total == 0) return cudaSuccess;
    int64_t blocks = cdiv(total, 256);
    const int64_t cap = (int64_t)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    if (chunk) im2row_kernel<T, true><<<(unsigned)blocks, 256, 0, s>>>(cv, pixels, (const T*)X, (T*)out, ld);
    else im2row_kernel<T, false><<<(unsigned)blocks, 256, 0, s>>>(cv, pixels, (const T*)X, (T*)out, ld);
    return cudaGetLastError();
}

static cudaError_t launch_im2row(int dtype, const ConvIndex& cv, int64_t pixels, const void* X, void* out, int64_t ld,
                                 cudaStream_t s) {
    // 16-bit values are moved as bit patterns: the transform never converts
    return dtype == GEMM_F32 ? launch_im2row_t<float>(cv, pixels, X, out, ld, s)
                             : launch_im2row_t<unsigned short>(cv, pixels, X, out, ld, s);
}

// ---- validation shared by the entry points: fills the index map; returns 0 or the negative argument position
static int conv_setup(int dtype, const conv_shape_t* sh, const void* X, ConvIndex* cv, int64_t* m, int64_t* n, int64_t* k) {
    if (dtype != GEMM_F32 && dtype != GEMM_F16 && dtype != GEMM_BF16) return -1;
    if (sh == nullptr) return -2;
    if (sh->batch < 0 || sh->h < 1 || sh->w < 1 || sh->c_in < 1 || sh->c_out < 0 || sh->kh < 1 || sh->kw < 1 ||
        sh->stride_h < 1 || sh->stride_w < 1 || sh->pad_h < 0 || sh->pad_w < 0)
        return -2;
    if (sh->h + 2 * (int64_t)sh->pad_h < sh->kh || sh->w + 2 * (int64_t)sh->pad_w < sh->kw) return -2;
    const int64_t ho = (sh->h + 2 * (int64_t)sh->pad_h - sh->kh) / sh->stride_h + 1;
    const int64_t wo = (sh->w + 2 * (int64_t)sh->pad_w - sh->kw) / sh->stride_w + 1;
    // 32-bit pixel arithmetic inside the kernels
    if (sh->h > 0x3FFFFFFF || sh->w > 0x3FFFFFFF || ho * wo > 0x7FFFFFFF || sh->batch > 0x7FFFFFFF ||
        (int64_t)sh->kh * sh->kw > 0x7FFF)
        return -2;
    cv->X = X;
    cv->h = sh->h; cv->w = sh->w; cv->c_in = sh->c_in;
    cv->ho = (int32_t)ho; cv->wo = (int32_t)wo;
    cv->kh = sh->kh; cv->kw = sh->kw; cv->sh = sh->stride_h; cv->sw = sh->stride_w; cv->ph = sh->pad_h; cv->pw = sh->pad_w;
    *m = sh->c_out;
    *n = sh->batch * ho * wo;
    *k = (int64_t)sh->kh * sh->kw * sh->c_in;
    return 0;
}

static bool lowering_is_identity(const ConvIndex& cv) {
    return cv.kh == 1 && cv.kw == 1 && cv.sh == 1 && cv.sw == 1 && cv.ph == 0 && cv.pw == 0;
}

// can the kernels read L through the index map for this call?
static bool fused_possible(int dtype, const ConvIndex& cv, int64_t batch, const void* W, int64_t ldw) {
    if (dtype == GEMM_F32) return true;
    const bool w_ok = (reinterpret_cast<uintptr_t>(W) & 15) == 0 && ldw % 8 == 0;      // the filter matrix goes through TMA as it is
    return w_ok && conv_tma_eligible(dtype, cv, batch);
}

}  // namespace b200gemm

using namespace b200gemm;

extern "C" {

int conv2d_force_lowering(int how) {
    if (how != 0 && how != CONV_LOWERING_FUSED && how != CONV_LOWERING_EXPLICIT) return -1;
    g_force_lowering = how;
    return GEMM_OK;
}

int im2row(int dtype, const conv_shape_t* shape, const void* X, void* out, int64_t ld, void* stream) {
    ConvIndex cv;
    int64_t m, n, k;
    const int bad = conv_setup(dtype, shape, X, &cv, &m, &n, &k);
    if (bad) return bad;
    if (n == 0) return GEMM_OK;
    const int es = elem_size(dtype);
    if (X == nullptr || (reinterpret_cast<uintptr_t>(X) % es) != 0) return -3;
    if (out == nullptr || (reinterpret_cast<uintptr_t>(out) % es) != 0) return -4;
    if (ld < k) return -5;
    const cudaError_t e = launch_im2row(dtype, cv, n, X, out, ld, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { note_launch_error(e); return GEMM_ERR_LAUNCH; }
    return GEMM_OK;
}

size_t conv2d_workspace_bytes(int dtype, const conv_shape_t* shape) {
    ConvIndex cv;
    int64_t m, n, k;
    if (conv_setup(dtype, shape, reinterpret_cast<const void*>(16), &cv, &m, &n, &k) != 0) return 0;
    if (m == 0 || n == 0) return 0;
    size_t need = gemm_workspace_bytes(dtype, 'N', 'N', m, n, k);
    if (lowering_is_identity(cv)) return need;
    // judged for 16-byte aligned tensors and a filter matrix TMA can address
    const bool fused = fused_possible(dtype, cv, shape->batch, reinterpret_cast<const void*>(16), 8);
    if (!fused || g_force_lowering == CONV_LOWERING_EXPLICIT) need += (size_t)rup(rup(k, 8) * n * elem_size(dtype), 256);
    return need;
}

int conv2d_im2row(int dtype, const conv_shape_t* shape, float alpha, const void* X, const void* W, int64_t ldw,
                  float beta, void* Y, int64_t ldy, void* stream) {
    ConvIndex cv;
    int64_t m, n, k;
    const int bad = conv_setup(dtype, shape, X, &cv, &m, &n, &k);
    if (bad) return bad;
    const int es = elem_size(dtype);
    const bool needs_ab = m > 0 && n > 0 && alpha != 0.0f;
    if (needs_ab && X == nullptr) return -4;
    if (X != nullptr && (reinterpret_cast<uintptr_t>(X) % es) != 0) return -4;
    if (needs_ab && W == nullptr) return -5;
    if (W != nullptr && (reinterpret_cast<uintptr_t>(W) % es) != 0) return -5;
    if (ldw < (m > 1 ? m : 1)) return -6;
    if (m > 0 && n > 0 && Y == nullptr) return -8;
    if (Y != nullptr && (reinterpret_cast<uintptr_t>(Y) % 4) != 0) return -8;
    if (ldy < (m > 1 ? m : 1)) return -9;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    if (m == 0 || n == 0 || alpha == 0.0f || lowering_is_identity(cv)) {
        // nothing to lower: scaling-only cases and 1 x 1 layers, whose lowered matrix is the NHWC tensor itself
        const int rc = gemm(dtype, 'N', 'N', m, n, k, alpha, W, ldw, X, cv.c_in, beta, Y, ldy, stream);
        if (rc == GEMM_OK) note_lowering(CONV_LOWERING_IDENTITY);
        return rc;
    }

    GemmArgs a{dtype, false, false, m, n, k, alpha, beta, W, nullptr, static_cast<float*>(Y), ldw, k, ldy, s, nullptr};
    const bool can_fuse = fused_possible(dtype, cv, shape->batch, W, ldw);
    const bool fuse = can_fuse && g_force_lowering != CONV_LOWERING_EXPLICIT;
    if (fuse) {
        a.conv = &cv;
        const int rc = dispatch_gemm(a, 0);
        if (rc == GEMM_OK) note_lowering(CONV_LOWERING_FUSED);
        return rc;
    }

    // explicit route: L goes to the head of the workspace (leading dimension a multiple of 8 elements so that TMA
    // can address it), the GEMM uses what is left
    void* ws = nullptr;
    size_t ws_bytes = 0;
    if (!registered_workspace(&ws, &ws_bytes)) return GEMM_ERR_LAUNCH;
    const int64_t ld = rup(k, 8);
    const size_t l_bytes = (size_t)rup(ld * n * es, 256);
    if (ws == nullptr || ws_bytes < l_bytes) return GEMM_ERR_WORKSPACE;
    const cudaError_t e = launch_im2row(dtype, cv, n, X, ws, ld, s);
    if (e != cudaSuccess) { note_launch_error(e); return GEMM_ERR_LAUNCH; }
    a.B = ws;
    a.ldb = ld;
    const int rc = dispatch_gemm(a, l_bytes);
    if (rc == GEMM_OK) note_lowering(CONV_LOWERING_EXPLICIT);
    return rc;
}

}  // extern "C"
