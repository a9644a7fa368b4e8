// Generic SIMT GEMM (any dtype, transpose flag, alignment and leading dimension), the C <- beta*C
// kernel and the split-k reduction.  These are the correctness anchors: every load and store is
// bounds-checked and scalar.
#include "internal.cuh"

namespace b200gemm {

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__half>(__half v) { return __half2float(v); }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

// Epilogue of Fig. 3 in BLAS form: alpha*acc + beta*C0, C0 untouched when beta == 0.
__device__ __forceinline__ float epilogue(float alpha, float acc, float beta, const float* c) {
    float r = alpha * acc;
    if (beta != 0.0f) r = fmaf(beta, *c, r);
    return r;
}
// the same on element i of a C that may be 16-bit: one rounding to the result type at the store
__device__ __forceinline__ void epilogue_store(float alpha, float acc, float beta, float* C, int out16, int64_t i) {
    float r = alpha * acc;
    if (beta != 0.0f) r = fmaf(beta, load_c(C, out16, i), r);
    store_c(C, out16, i, r);
}

constexpr int GT = 64;   // CTA tile (GT x GT) of C
constexpr int GK = 16;   // k extent of one shared-memory stage

// 256 threads; thread (tx, ty) owns the 4x4 entries (tx + 16 i, ty + 16 j) of the tile.
template <typename T, bool TA, bool TB>
__global__ void __launch_bounds__(256)
simt_generic_kernel(int64_t m, int64_t n, int64_t k, float alpha, const T* __restrict__ A, int64_t lda,
                    const T* __restrict__ B, int64_t ldb, float beta, float* __restrict__ C, int64_t ldc,
                    int64_t tiles_m, int out16, int64_t strideA, int64_t strideB, int64_t strideC) {
    __shared__ float As[GK][GT + 1];
    __shared__ float Bs[GK][GT + 1];
    // strided batch: blockIdx.y is the problem; strideC counts elements of C's type
    A += (int64_t)blockIdx.y * strideA;
    B += (int64_t)blockIdx.y * strideB;
    C = out16 ? reinterpret_cast<float*>(reinterpret_cast<uint16_t*>(C) + (int64_t)blockIdx.y * strideC)
              : C + (int64_t)blockIdx.y * strideC;
    const int t = threadIdx.x;
    const int tx = t & 15, ty = t >> 4;
    const int64_t tile = blockIdx.x;
    const int64_t i0 = (tile % tiles_m) * GT, j0 = (tile / tiles_m) * GT;

    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

    for (int64_t k0 = 0; k0 < k; k0 += GK) {
#pragma unroll
        for (int e = 0; e < (GT * GK) / 256; ++e) {
            int idx = t + e * 256;
            // A: walk the contiguous dimension of the stored matrix with consecutive threads
            int mm = TA ? idx / GK : idx % GT;
            int kk = TA ? idx % GK : idx / GT;
            int64_t gi = i0 + mm, gk = k0 + kk;
            float v = 0.0f;
            if (gi < m && gk < k) v = to_float<T>(TA ? A[gk + gi * lda] : A[gi + gk * lda]);
            As[kk][mm] = v;
            int nn = TB ? idx % GT : idx / GK;
            int kb = TB ? idx / GT : idx % GK;
            int64_t gj = j0 + nn;
            gk = k0 + kb;
            v = 0.0f;
            if (gj < n && gk < k) v = to_float<T>(TB ? B[gj + gk * ldb] : B[gk + gj * ldb]);
            Bs[kb][nn] = v;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < GK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][tx + 16 * i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][ty + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        int64_t gj = j0 + ty + 16 * j;
        if (gj >= n) continue;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int64_t gi = i0 + tx + 16 * i;
            if (gi < m) epilogue_store(alpha, acc[i][j], beta, C, out16, gi + gj * ldc);
        }
    }
}

template <typename T>
static cudaError_t launch_generic_t(const GemmArgs& a, int64_t sA, int64_t sB, int64_t sC, int64_t batch) {
    int64_t tiles_m = (a.m + GT - 1) / GT, tiles_n = (a.n + GT - 1) / GT;
    int64_t tiles = tiles_m * tiles_n;
    if (tiles > 0x7FFFFFFFLL || batch < 1 || batch > 65535) return cudaErrorInvalidConfiguration;
    dim3 grid((unsigned)tiles, (unsigned)batch), block(256);
    const T* A = (const T*)a.A;
    const T* B = (const T*)a.B;
#define LAUNCH(TA_, TB_)                                                                              \
    simt_generic_kernel<T, TA_, TB_><<<grid, block, 0, a.stream>>>(a.m, a.n, a.k, a.alpha, A, a.lda, B, \
                                                                   a.ldb, a.beta, a.C, a.ldc, tiles_m, a.out16, sA, sB, sC)
    if (!a.ta && !a.tb) LAUNCH(false, false);
    else if (a.ta && !a.tb) LAUNCH(true, false);
    else if (!a.ta && a.tb) LAUNCH(false, true);
    else LAUNCH(true, true);
#undef LAUNCH
    return cudaGetLastError();
}

cudaError_t launch_simt_generic(const GemmArgs& a, gemm_config_t* cfg, int64_t strideA, int64_t strideB, int64_t strideC,
                                int64_t batch) {
    cfg->kernel = GEMM_KERNEL_SIMT_GENERIC;
    cfg->tile_m = GT; cfg->tile_n = GT; cfg->tile_k = GK; cfg->split_k = 1; cfg->stages = 1;
    cfg->grid = (int32_t)(((a.m + GT - 1) / GT) * ((a.n + GT - 1) / GT));
    cfg->vector_a = cfg->vector_b = 1;
    cfg->launches = 1;
    if (a.dtype == GEMM_F32) return launch_generic_t<float>(a, strideA, strideB, strideC, batch);
    if (a.dtype == GEMM_F16) return launch_generic_t<__half>(a, strideA, strideB, strideC, batch);
    return launch_generic_t<__nv_bfloat16>(a, strideA, strideB, strideC, batch);
}

// ---------------------------------------------------------------- C <- beta*C

__global__ void __launch_bounds__(256)
scale_kernel(int64_t m, int64_t n, float beta, float* __restrict__ C, int64_t ldc, int out16, int64_t strideC) {
    C = out16 ? reinterpret_cast<float*>(reinterpret_cast<uint16_t*>(C) + (int64_t)blockIdx.z * strideC)
              : C + (int64_t)blockIdx.z * strideC;
    for (int64_t j = blockIdx.y; j < n; j += gridDim.y)
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < m; i += (int64_t)gridDim.x * blockDim.x) {
            const int64_t e = i + j * ldc;
            store_c(C, out16, e, (beta == 0.0f) ? 0.0f : beta * load_c(C, out16, e));
        }
}

cudaError_t launch_scale(const GemmArgs& a, int64_t strideC, int64_t batch) {
    if (batch < 1 || batch > 65535) return cudaErrorInvalidConfiguration;
    unsigned gx = (unsigned)((a.m + 255) / 256 > 1024 ? 1024 : (a.m + 255) / 256);
    unsigned gy = (unsigned)(a.n > 32768 ? 32768 : a.n);
    scale_kernel<<<dim3(gx, gy, (unsigned)batch), 256, 0, a.stream>>>(a.m, a.n, a.beta, a.C, a.ldc, a.out16, strideC);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- split-k reduction + epilogue

// partials: [split][n][m] fp32 (leading dimension m).  Summed in increasing split index (deterministic).
// Thread block 32 x 8: x walks rows (V of them per thread), y walks columns.
template <int V>
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(int64_t m, int64_t n, int splits, const float* __restrict__ partials, float alpha, float beta,
                     float* __restrict__ C, int64_t ldc, int out16) {
    const int64_t plane = m * n;
    const int64_t mv = m / V;
    for (int64_t j = (int64_t)blockIdx.y * blockDim.y + threadIdx.y; j < n; j += (int64_t)gridDim.y * blockDim.y)
        for (int64_t iv = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; iv < mv; iv += (int64_t)gridDim.x * blockDim.x) {
            const float* p = partials + iv * V + j * m;
            float* c = C + iv * V + j * ldc;
            if (V == 4) {
                float4 s = *reinterpret_cast<const float4*>(p);
                for (int z = 1; z < splits; ++z) {
                    const float4 q = *reinterpret_cast<const float4*>(p + (int64_t)z * plane);
                    s.x += q.x; s.y += q.y; s.z += q.z; s.w += q.w;
                }
                float4 r = make_float4(alpha * s.x, alpha * s.y, alpha * s.z, alpha * s.w);
                if (beta != 0.0f) {
                    const float4 c0 = *reinterpret_cast<const float4*>(c);
                    r.x = fmaf(beta, c0.x, r.x); r.y = fmaf(beta, c0.y, r.y);
                    r.z = fmaf(beta, c0.z, r.z); r.w = fmaf(beta, c0.w, r.w);
                }
                *reinterpret_cast<float4*>(c) = r;
            } else {
                float s = *p;
                for (int z = 1; z < splits; ++z) s += p[(int64_t)z * plane];
                epilogue_store(alpha, s, beta, C, out16, iv + j * ldc);
            }
        }
}

cudaError_t launch_splitk_reduce(const GemmArgs& a, int splits, const float* partials) {
    const bool vec = a.out16 == 0 && a.m % 4 == 0 && a.ldc % 4 == 0 && (reinterpret_cast<uintptr_t>(partials) & 15) == 0 &&
                     (reinterpret_cast<uintptr_t>(a.C) & 15) == 0;       // 128-bit path: fp32 results only
    const int64_t mv = vec ? a.m / 4 : a.m;
    int64_t gx = (mv + 31) / 32, gy = (a.n + 7) / 8;
    if (gx > 1024) gx = 1024;
    if (gy > 32768) gy = 32768;
    dim3 grid((unsigned)gx, (unsigned)gy), block(32, 8);
    if (vec) splitk_reduce_kernel<4><<<grid, block, 0, a.stream>>>(a.m, a.n, splits, partials, a.alpha, a.beta, a.C, a.ldc, a.out16);
    else splitk_reduce_kernel<1><<<grid, block, 0, a.stream>>>(a.m, a.n, splits, partials, a.alpha, a.beta, a.C, a.ldc, a.out16);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- 16-bit operand repack (aligned leading dimension)

// One thread per 16-byte chunk (8 elements) of the aligned copy.  A chunk that lies wholly inside its column is read
// as 32-bit words: four when its first source element sits on a 4-byte boundary, otherwise five, shifted by one
// element with byte permutes (columns of odd length alternate between the two cases).  Chunks at the end of a column,
// the last column (whose fifth word could lie beyond the matrix) and the very first chunk go element by element; rows rows..ld_out-1 of
// the copy are zero.
__global__ void __launch_bounds__(256)
repack16_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t cols, int64_t ld, uint16_t* __restrict__ dst,
                int64_t ld_out) {
    const int64_t chunks = ld_out / 8;                      // per column (ld_out is a multiple of 8)
    const int64_t total = chunks * cols;
    for (int64_t u = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; u < total; u += (int64_t)gridDim.x * blockDim.x) {
        const int64_t j = u / chunks, i0 = (u - j * chunks) * 8;
        const uint16_t* sp = src + j * ld + i0;
        uint4 out;
        if (i0 + 8 <= rows && j + 1 < cols && u > 0) {      // (u == 0: the word below the first element may lie before the matrix)
            const uintptr_t addr = reinterpret_cast<uintptr_t>(sp);
            const uint32_t* w = reinterpret_cast<const uint32_t*>(addr & ~(uintptr_t)3);
            if ((addr & 2) == 0) {
                out = make_uint4(__ldg(w), __ldg(w + 1), __ldg(w + 2), __ldg(w + 3));
            } else {                                        // the chunk starts in the upper half of w[0]
                const uint32_t a = __ldg(w), b = __ldg(w + 1), c = __ldg(w + 2), d = __ldg(w + 3), e = __ldg(w + 4);
                out = make_uint4(__byte_perm(a, b, 0x5432), __byte_perm(b, c, 0x5432), __byte_perm(c, d, 0x5432),
                                 __byte_perm(d, e, 0x5432));
            }
        } else {
            uint32_t h[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) h[t] = (i0 + t < rows) ? (uint32_t)sp[t] : 0u;
            out = make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
        }
        *reinterpret_cast<uint4*>(dst + j * ld_out + i0) = out;
    }
}

cudaError_t launch_repack16(const void* src, int64_t rows, int64_t cols, int64_t ld, void* dst, int64_t ld_out,
                            cudaStream_t stream) {
    const int64_t total = (ld_out / 8) * cols;
    if (total <= 0) return cudaSuccess;
    int64_t blocks = (total + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    repack16_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const uint16_t*)src, rows, cols, ld, (uint16_t*)dst, ld_out);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- fp32 -> three bfloat16 pieces

// One thread per four consecutive rows of a column.  Each piece is rounded to nearest even from what the earlier
// pieces left over; the subtractions are exact in fp32 (the piece shares the leading bits of what it was rounded from).
__global__ void __launch_bounds__(256)
split3_kernel(const float* __restrict__ src, int64_t rows, int64_t cols, int64_t ld, __nv_bfloat16* __restrict__ p1,
              __nv_bfloat16* __restrict__ p2, __nv_bfloat16* __restrict__ p3, int64_t ld_p, int vec, int64_t rows_out,
              int64_t cols_out) {
    // rows_out (a multiple of 4) x cols_out entries of every piece are written: zeros beyond the rows x cols of the source
    const int64_t quads = rows_out / 4;
    for (int64_t j = blockIdx.y; j < cols_out; j += gridDim.y)
        for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q < quads; q += (int64_t)gridDim.x * blockDim.x) {
            const int64_t i = q * 4;
            float x[4] = {0.f, 0.f, 0.f, 0.f};
            if (j < cols && i < rows) {
                const float* s = src + i + j * ld;
                if (vec && i + 3 < rows) {
                    const float4 v = __ldg(reinterpret_cast<const float4*>(s));
                    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (i + e < rows) x[e] = __ldg(s + e);
                }
            }
            uint16_t h[3][4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float r = x[e];
#pragma unroll
                for (int t = 0; t < 3; ++t) {
                    const __nv_bfloat16 b = __float2bfloat16_rn(r);
                    h[t][e] = __bfloat16_as_ushort(b);
                    r -= __bfloat162float(b);
                }
            }
            // ld_p is a multiple of 8 and the pieces are 16-byte aligned: the four values of a piece go out as one 8-byte store
            __nv_bfloat16* out[3] = {p1, p2, p3};
#pragma unroll
            for (int t = 0; t < 3; ++t) {
                const uint2 w = make_uint2((uint32_t)h[t][0] | ((uint32_t)h[t][1] << 16), (uint32_t)h[t][2] | ((uint32_t)h[t][3] << 16));
                *reinterpret_cast<uint2*>(out[t] + i + j * ld_p) = w;
            }
        }
}

// rows_out / cols_out: the extent written per piece (0 = the source's own, rows rounded up to 4); ld_p >= rows_out
cudaError_t launch_split3(const float* src, int64_t rows, int64_t cols, int64_t ld, void* p1, void* p2, void* p3,
                          int64_t ld_p, cudaStream_t stream, int64_t rows_out, int64_t cols_out) {
    if (rows == 0 || cols == 0) return cudaSuccess;
    if (rows_out == 0) rows_out = (rows + 3) / 4 * 4;
    if (cols_out == 0) cols_out = cols;
    if (rows_out % 4 != 0 || rows_out < rows || cols_out < cols || ld_p < rows_out) return cudaErrorInvalidValue;
    const int64_t quads = rows_out / 4;
    int64_t gx = (quads + 255) / 256, gy = cols_out;
    if (gx > 1024) gx = 1024;
    if (gy > 32768) gy = 32768;
    const int vec = ((reinterpret_cast<uintptr_t>(src) & 15) == 0 && ld % 4 == 0) ? 1 : 0;
    split3_kernel<<<dim3((unsigned)gx, (unsigned)gy), 256, 0, stream>>>(src, rows, cols, ld, (__nv_bfloat16*)p1, (__nv_bfloat16*)p2,
                                                                     (__nv_bfloat16*)p3, ld_p, vec, rows_out, cols_out);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- tail reduction

// One block row per tail tile (blockIdx.x) and a quarter of its entries per blockIdx.y: sums the tile's k ranges in
// increasing order (deterministic) and applies alpha / beta once.
__global__ void __launch_bounds__(256)
tail_reduce_kernel(int64_t m, int64_t n, float alpha, float beta, float* __restrict__ C, int64_t ldc, int tiles_m,
                   int tiles_n, int bm, int bn, int group, TailSplit tail) {
    const int tl = blockIdx.x;
    int tm, tn;
    decode_tile(tail.first + tl, tiles_m, tiles_n, &tm, &tn, group);
    const int64_t i0 = (int64_t)tm * bm, j0 = (int64_t)tn * bn;
    const int tile_elems = bm * bn;
    const float* slot = tail.partials + (int64_t)tl * tail.splits * tile_elems;
    const int vecs = tile_elems / 4, per_y = (vecs + gridDim.y - 1) / gridDim.y;
    const int v_end = min(vecs, (int)(blockIdx.y + 1) * per_y);
    for (int v = blockIdx.y * per_y + threadIdx.x; v < v_end; v += blockDim.x) {
        const int e = v * 4, r = e % bm, c = e / bm;
        float4 s4 = *reinterpret_cast<const float4*>(slot + e);
        for (int z = 1; z < tail.splits; ++z) {
            const float4 q = *reinterpret_cast<const float4*>(slot + (int64_t)z * tile_elems + e);
            s4.x += q.x; s4.y += q.y; s4.z += q.z; s4.w += q.w;
        }
        const int64_t gi = i0 + r, gj = j0 + c;
        if (gj >= n) continue;
        const float sv[4] = {s4.x, s4.y, s4.z, s4.w};
        float* cp = C + gi + gj * ldc;
#pragma unroll
        for (int q = 0; q < 4; ++q)
            if (gi + q < m) {
                float o = alpha * sv[q];
                if (beta != 0.0f) o = fmaf(beta, cp[q], o);
                cp[q] = o;
            }
    }
}

cudaError_t launch_tail_reduce(const GemmArgs& a, int bm, int bn, int group, TailSplit tail) {
    const int64_t tiles_m = (a.m + bm - 1) / bm, tiles_n = (a.n + bn - 1) / bn;
    const int64_t tail_tiles = tiles_m * tiles_n - tail.first;
    if (tail_tiles <= 0) return cudaSuccess;
    tail_reduce_kernel<<<dim3((unsigned)tail_tiles, 4), 256, 0, a.stream>>>(a.m, a.n, a.alpha, a.beta, a.C, a.ldc,
                                                                           (int)tiles_m, (int)tiles_n, bm, bn, group, tail);
    return cudaGetLastError();
}

}  // namespace b200gemm
