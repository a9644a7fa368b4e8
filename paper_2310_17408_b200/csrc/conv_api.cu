// Convolution layers through the im2row lowering (Section IV-C): the front end that turns a layer into the GEMM
//     Y[C_out x pixels] = W[C_out x k] * L[k x pixels],   k = kh*kw*C_in,
// chooses how L comes to exist (fused into the GEMM kernels' operand staging, written out by im2row_kernel, or not
// needed at all), and the im2row transform itself as a kernel.
#include "internal.cuh"

namespace b200gemm {

static thread_local int g_force_lowering = 0;     // per host thread, like the other forcing knobs

static inline int64_t cdiv(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline int64_t rup(int64_t a, int64_t b) { return cdiv(a, b) * b; }

// ---- the transform as a copy kernel.  Column j of L is the patch of output pixel j: kh*kw runs of C_in contiguous
// elements of X (or zeros).  Three forms, by what the alignment allows:
//   MODE 0  one thread per 16-byte chunk, loaded and stored whole (C_in a multiple of the chunk, everything aligned)
//   MODE 1  one thread per 16-byte chunk of L, gathered element by element and stored whole (any C_in; L aligned);
//           rows k..ld-1 that fall into a chunk are written as zeros
//   MODE 2  one thread per element (no alignment at all)
// Idx: type of the flat work index (32-bit whenever the element count allows: the index is taken apart by divisions,
// and 64-bit divisions would cost more than the copy itself)
template <typename T, int MODE, typename Idx>
__global__ void __launch_bounds__(256)
im2row_kernel(const ConvIndex cv, int64_t pixels, int k, const T* __restrict__ X, T* __restrict__ out, int64_t ld) {
    constexpr int PER = MODE == 2 ? 1 : (int)(16 / sizeof(T));      // elements of L written by one thread
    const uint32_t cin = (uint32_t)cv.c_in, kw = (uint32_t)cv.kw;
    const uint32_t per_col = MODE == 1 ? (uint32_t)(ld / PER) : (uint32_t)(k / PER);     // threads per column of L
    const Idx total = (Idx)pixels * (Idx)per_col;
    const uint32_t hw = (uint32_t)(cv.ho * cv.wo);
    for (Idx idx = (Idx)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (Idx)gridDim.x * blockDim.x) {
        const Idx j = idx / (Idx)per_col;
        const uint32_t p0 = (uint32_t)(idx - j * (Idx)per_col) * PER;     // first row of L this thread writes
        const uint32_t b = (uint32_t)(j / (Idx)hw), rem = (uint32_t)(j - (Idx)b * (Idx)hw);
        const int oh = (int)(rem / (uint32_t)cv.wo), ow = (int)(rem - (uint32_t)oh * (uint32_t)cv.wo);
        const int h0 = oh * cv.sh - cv.ph, w0 = ow * cv.sw - cv.pw;
        const int64_t base = (((int64_t)b * cv.h + h0) * cv.w + w0) * cv.c_in;
        auto source = [&](uint32_t p, bool& inside) {      // element offset in X of row p of this column
            const uint32_t tap = p / cin, c = p - tap * cin;
            const int fr = (int)(tap / kw), fs = (int)(tap - (uint32_t)fr * kw);
            inside = p < (uint32_t)k && (unsigned)(h0 + fr) < (unsigned)cv.h && (unsigned)(w0 + fs) < (unsigned)cv.w;
            return base + ((int64_t)fr * cv.w + fs) * cv.c_in + c;
        };
        T* dst = out + (int64_t)j * ld + p0;
        if (MODE == 0) {
            bool inside;
            const int64_t src = source(p0, inside);
            *reinterpret_cast<uint4*>(dst) = inside ? __ldg(reinterpret_cast<const uint4*>(X + src)) : make_uint4(0, 0, 0, 0);
        } else if (MODE == 1) {
            // Inside one filter row r the k index runs over (s, c), which is also how the NHWC image row lies in
            // memory: the source of row p is rowbase(r) + q with q = p - r*kw*C_in, and the horizontal bounds become
            // a range of q.  One division for the chunk's first row; after that q and r walk forward.
            union { uint4 q; T e[PER]; } v;
            const uint32_t seg = kw * cin;                                       // elements per filter row
            uint32_t fr = p0 / seg, q = p0 - fr * seg;
            const uint32_t qlo = (uint32_t)max(0, -w0) * cin;
            const uint32_t qhi = (uint32_t)max(0, min((int)kw, (int)cv.w - w0)) * cin;
            const int64_t rowstep = cv.w * cv.c_in;
            int64_t rowbase = base + (int64_t)fr * rowstep;
#pragma unroll
            for (int i = 0; i < PER; ++i) {
                const bool inside = p0 + i < (uint32_t)k && (unsigned)(h0 + (int)fr) < (unsigned)cv.h && q >= qlo && q < qhi;
                v.e[i] = inside ? __ldg(X + rowbase + q) : T(0);
                if (++q == seg) { q = 0; ++fr; rowbase += rowstep; }
            }
            *reinterpret_cast<uint4*>(dst) = v.q;
        } else {
            bool inside;
            const int64_t src = source(p0, inside);
            *dst = inside ? __ldg(X + src) : T(0);
        }
    }
}

template <typename T>
static cudaError_t launch_im2row_t(const ConvIndex& cv, int64_t pixels, const void* X, void* out, int64_t ld, cudaStream_t s) {
    const int es = (int)sizeof(T);
    const int64_t k = (int64_t)cv.kh * cv.kw * cv.c_in;
    const bool out_ok = (ld * es) % 16 == 0 && (reinterpret_cast<uintptr_t>(out) & 15) == 0;
    const bool in_ok = (cv.c_in * es) % 16 == 0 && (reinterpret_cast<uintptr_t>(X) & 15) == 0;
    const int mode = out_ok ? (in_ok ? 0 : 1) : 2;
    const int64_t per = mode == 2 ? 1 : 16 / es;
    const int64_t total = pixels * (mode == 1 ? ld / per : k / per);
    if (total == 0) return cudaSuccess;
    int64_t blocks = cdiv(total, 256);
    const int64_t cap = (int64_t)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    const bool small = total + blocks * 256 < 0x7FFFFFFFLL && pixels < 0x7FFFFFFFLL;      // flat index and its stride fit 32 bits
#define IM2ROW_LAUNCH(MODE_, IDX_) \
    im2row_kernel<T, MODE_, IDX_><<<(unsigned)blocks, 256, 0, s>>>(cv, pixels, (int)k, (const T*)X, (T*)out, ld)
    if (small) {
        if (mode == 0) IM2ROW_LAUNCH(0, uint32_t);
        else if (mode == 1) IM2ROW_LAUNCH(1, uint32_t);
        else IM2ROW_LAUNCH(2, uint32_t);
    } else {
        if (mode == 0) IM2ROW_LAUNCH(0, int64_t);
        else if (mode == 1) IM2ROW_LAUNCH(1, int64_t);
        else IM2ROW_LAUNCH(2, int64_t);
    }
#undef IM2ROW_LAUNCH
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
    if (dtype != GEMM_F32 && dtype != GEMM_F16 && dtype != GEMM_BF16 && dtype != GEMM_F16_C16 && dtype != GEMM_BF16_C16)
        return -1;
    if (sh == nullptr) return -2;
    if (sh->batch < 0 || sh->h < 1 || sh->w < 1 || sh->c_in < 1 || sh->c_out < 0 || sh->kh < 1 || sh->kw < 1 ||
        sh->stride_h < 1 || sh->stride_w < 1 || sh->pad_h < 0 || sh->pad_w < 0)
        return -2;
    if (sh->h + 2 * (int64_t)sh->pad_h < sh->kh || sh->w + 2 * (int64_t)sh->pad_w < sh->kw) return -2;
    const int64_t ho = (sh->h + 2 * (int64_t)sh->pad_h - sh->kh) / sh->stride_h + 1;
    const int64_t wo = (sh->w + 2 * (int64_t)sh->pad_w - sh->kw) / sh->stride_w + 1;
    // 32-bit pixel arithmetic inside the kernels
    if (sh->h > 0x3FFFFFFF || sh->w > 0x3FFFFFFF || ho * wo > 0x7FFFFFFF || sh->batch > 0x7FFFFFFF ||
        (int64_t)sh->kh * sh->kw > 0x7FFF || (int64_t)sh->kh * sh->kw * sh->c_in > 0x7FFFFFFF)
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
    const cudaError_t e = launch_im2row(input_dtype(dtype), cv, n, X, out, ld, static_cast<cudaStream_t>(stream));
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
    const bool fused = fused_possible(input_dtype(dtype), cv, shape->batch, reinterpret_cast<const void*>(16), 8);
    const bool scalar_map = dtype == GEMM_F32 && cv.c_in % 4 != 0;       // served faster by writing L first
    if (!fused || scalar_map || g_force_lowering == CONV_LOWERING_EXPLICIT)
        need += (size_t)rup(rup(k, 8) * n * elem_size(dtype), 256);
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
    if (Y != nullptr && (reinterpret_cast<uintptr_t>(Y) % c_elem_size(dtype)) != 0) return -8;
    if (ldy < (m > 1 ? m : 1)) return -9;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    if (m == 0 || n == 0 || alpha == 0.0f || lowering_is_identity(cv)) {
        // nothing to lower: scaling-only cases and 1 x 1 layers, whose lowered matrix is the NHWC tensor itself
        // (in the scaling-only cases the operands are not read; the leading dimension only has to be a legal one)
        const int rc = gemm(dtype, 'N', 'N', m, n, k, alpha, W, ldw, X, lowering_is_identity(cv) ? cv.c_in : k, beta, Y, ldy, stream);
        if (rc == GEMM_OK) note_lowering(CONV_LOWERING_IDENTITY);
        return rc;
    }

    GemmArgs a{input_dtype(dtype), false, false, m, n, k, alpha, beta, W, nullptr, static_cast<float*>(Y), ldw, k, ldy, s, nullptr};
    a.out16 = output16(dtype);
    const bool can_fuse = fused_possible(input_dtype(dtype), cv, shape->batch, W, ldw);
    void* ws = nullptr;
    size_t ws_bytes = 0;
    if (!registered_workspace(s, &ws, &ws_bytes)) return GEMM_ERR_LAUNCH;
    const int64_t ld = rup(k, 8);
    const size_t l_bytes = (size_t)rup(ld * n * es, 256);
    const bool room = ws != nullptr && ws_bytes >= l_bytes;
    // fp32 layers whose channel count rules out 128-bit loads (the 3-channel first layers) run the index map with
    // scalar loads at about a third of the kernel's speed: writing L first is faster when there is room for it
    const bool scalar_map = dtype == GEMM_F32 && (cv.c_in % 4 != 0 || (reinterpret_cast<uintptr_t>(X) & 15) != 0);
    bool fuse = can_fuse && g_force_lowering != CONV_LOWERING_EXPLICIT;
    if (fuse && scalar_map && room && g_force_lowering != CONV_LOWERING_FUSED) fuse = false;
    if (fuse) {
        a.conv = &cv;
        const int rc = dispatch_gemm(a, 0);
        if (rc == GEMM_OK) note_lowering(CONV_LOWERING_FUSED);
        return rc;
    }

    // explicit route: L goes to the head of the workspace (leading dimension a multiple of 8 elements so that TMA
    // can address it), the GEMM uses what is left
    if (!room) {
        if (!can_fuse) return GEMM_ERR_WORKSPACE;
        a.conv = &cv;                               // forced explicit but no room: the fused route still works
        const int rc = dispatch_gemm(a, 0);
        if (rc == GEMM_OK) note_lowering(CONV_LOWERING_FUSED);
        return rc;
    }
    const cudaError_t e = launch_im2row(input_dtype(dtype), cv, n, X, ws, ld, s);
    if (e != cudaSuccess) { note_launch_error(e); return GEMM_ERR_LAUNCH; }
    a.B = ws;
    a.ldb = ld;
    const int rc = dispatch_gemm(a, l_bytes);
    if (rc == GEMM_OK) note_lowering(CONV_LOWERING_EXPLICIT);
    return rc;
}

}  // extern "C"
