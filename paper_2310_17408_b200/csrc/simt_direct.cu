// fp32 GEMM for tiny problems without operand staging: the counterpart of the paper's non-packed micro-kernel
// variant (Section III-B, "Edge Cases": for small problems packing does not pay, so the kernel reads A where it
// lies).  Every thread owns a 4 x 4 block of C and reads its four rows of op(A) and four columns of op(B) straight
// from global memory into registers (128-bit loads through the read-only path where alignment allows; L1 serves
// the reuse between neighbouring threads).  No shared memory, no barrier, no workspace, no reduction pass: one
// launch whose length is one thread's k loop, which is what matters when the whole problem is a few microseconds
// of work.  The unit of work is a 32 x 16 slab of one problem's C, one warp each; the slabs of all problems of a
// strided batch are numbered through, so that small problems share CTAs instead of leaving warps idle.
#include "internal.cuh"

namespace b200gemm {

constexpr int DT = 4;                 // thread tile (DT x DT)
constexpr int D_WARP_M = 8;           // threads of a warp along m (x 4 along n): a warp covers a 32 x 16 slab of C
constexpr int D_WARPS = 4;            // warps per CTA; every warp takes the next slab of the whole batch
constexpr int D_TILE_M = D_WARP_M * DT, D_TILE_N = 4 * DT;      // slab extents

// four consecutive k of one row (KCONT) or four consecutive rows at one k (!KCONT) of a stored matrix
template <bool VEC>
__device__ __forceinline__ void load4(const float* __restrict__ p, int64_t step, bool ok0, bool ok1, bool ok2, bool ok3,
                                      float (&v)[4]) {
    if (VEC) {      // step == 1, 16-byte aligned, all four in range
        const float4 q = __ldg(reinterpret_cast<const float4*>(p));
        v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
    } else {
        v[0] = ok0 ? __ldg(p) : 0.0f;
        v[1] = ok1 ? __ldg(p + step) : 0.0f;
        v[2] = ok2 ? __ldg(p + 2 * step) : 0.0f;
        v[3] = ok3 ? __ldg(p + 3 * step) : 0.0f;
    }
}

// TA / TB: op(X) = X^T.  VEC: pointers 16-byte aligned, leading dimensions and batch strides multiples of 4.
template <bool TA, bool TB, bool VEC>
__global__ void __launch_bounds__(32 * D_WARPS)
simt_direct_kernel(int64_t m, int64_t n, int64_t k, float alpha, const float* __restrict__ A, int64_t lda, int64_t strideA,
                   const float* __restrict__ B, int64_t ldb, int64_t strideB, float beta, float* __restrict__ C,
                   int64_t ldc, int64_t strideC, int tiles_m, int64_t slabs_per_problem, int64_t total_slabs) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t slab = (int64_t)blockIdx.x * D_WARPS + warp;
    const int64_t problem = slab / slabs_per_problem, within = slab - problem * slabs_per_problem;
    const int64_t tm = within % tiles_m, tn = within / tiles_m;
    const int64_t i0 = tm * D_TILE_M + (lane % D_WARP_M) * DT;
    const int64_t j0 = tn * D_TILE_N + (lane / D_WARP_M) * DT;
    A += problem * strideA;
    B += problem * strideB;
    C += problem * strideC;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (slab >= total_slabs || i0 >= m || j0 >= n) return;

    float acc[DT][DT];      // [column][row]
#pragma unroll
    for (int j = 0; j < DT; ++j)
#pragma unroll
        for (int i = 0; i < DT; ++i) acc[j][i] = 0.0f;
    const bool rows_in = i0 + DT <= m, cols_in = j0 + DT <= n;

    // Interior, aligned blocks take k sixteen at a time: all 32 128-bit loads of a round are issued before the first
    // product, so that a round costs one memory latency (the length of this loop is what the kernel is timed by).
    int64_t kdone = 0;
    if (VEC && rows_in && cols_in) {
        for (; kdone + 16 <= k; kdone += 16) {
            float4 av[16], bv[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                // !TA: av[u] = rows i0..i0+3 at k = kdone + u;   TA: av[u] = row i0 + u/4 at k = kdone + 4*(u%4) .. +3
                const float* pa = TA ? A + kdone + 4 * (u & 3) + (i0 + (u >> 2)) * lda : A + i0 + (kdone + u) * lda;
                // !TB: bv[u] = column j0 + u/4 at k = kdone + 4*(u%4) .. +3;   TB: bv[u] = columns j0..j0+3 at k = kdone + u
                const float* pb = TB ? B + j0 + (kdone + u) * ldb : B + kdone + 4 * (u & 3) + (j0 + (u >> 2)) * ldb;
                av[u] = __ldg(reinterpret_cast<const float4*>(pa));
                bv[u] = __ldg(reinterpret_cast<const float4*>(pb));
            }
            auto comp = [](const float4& v, int c) { return c == 0 ? v.x : (c == 1 ? v.y : (c == 2 ? v.z : v.w)); };
#pragma unroll
            for (int kk = 0; kk < 16; ++kk)      // increasing k, as everywhere
#pragma unroll
                for (int j = 0; j < DT; ++j) {
                    const float bj = TB ? comp(bv[kk], j) : comp(bv[j * 4 + (kk >> 2)], kk & 3);
#pragma unroll
                    for (int i = 0; i < DT; ++i) {
                        const float ai = TA ? comp(av[i * 4 + (kk >> 2)], kk & 3) : comp(av[kk], i);
                        acc[j][i] = fmaf(ai, bj, acc[j][i]);
                    }
                }
        }
    }

    // the rest (edge blocks, unaligned operands, the last k): steps of four, every element guarded.
    // a[kk][i] = op(A)(i0 + i, k0 + kk), b[kk][j] = op(B)(k0 + kk, j0 + j).
    for (int64_t k0 = kdone; k0 < k; k0 += 4) {
        float a[4][DT], b[4][DT];
        const bool k_in = k0 + 4 <= k;
        if (!TA) {      // stored m x k: four rows of one k are contiguous
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                float v[4];
                const bool kv = k0 + kk < k;
                const float* p = A + i0 + (k0 + kk) * lda;
                if (VEC && rows_in && kv) load4<true>(p, 1, true, true, true, true, v);
                else load4<false>(p, 1, kv && i0 < m, kv && i0 + 1 < m, kv && i0 + 2 < m, kv && i0 + 3 < m, v);
#pragma unroll
                for (int i = 0; i < DT; ++i) a[kk][i] = v[i];
            }
        } else {        // stored k x m: four k of one row are contiguous
#pragma unroll
            for (int i = 0; i < DT; ++i) {
                float v[4];
                const bool iv = i0 + i < m;
                const float* p = A + k0 + (i0 + i) * lda;
                if (VEC && k_in && iv) load4<true>(p, 1, true, true, true, true, v);
                else load4<false>(p, 1, iv && k0 < k, iv && k0 + 1 < k, iv && k0 + 2 < k, iv && k0 + 3 < k, v);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) a[kk][i] = v[kk];
            }
        }
        if (!TB) {      // stored k x n: four k of one column are contiguous
#pragma unroll
            for (int j = 0; j < DT; ++j) {
                float v[4];
                const bool jv = j0 + j < n;
                const float* p = B + k0 + (j0 + j) * ldb;
                if (VEC && k_in && jv) load4<true>(p, 1, true, true, true, true, v);
                else load4<false>(p, 1, jv && k0 < k, jv && k0 + 1 < k, jv && k0 + 2 < k, jv && k0 + 3 < k, v);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) b[kk][j] = v[kk];
            }
        } else {        // stored n x k: four columns of one k are contiguous
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                float v[4];
                const bool kv = k0 + kk < k;
                const float* p = B + j0 + (k0 + kk) * ldb;
                if (VEC && cols_in && kv) load4<true>(p, 1, true, true, true, true, v);
                else load4<false>(p, 1, kv && j0 < n, kv && j0 + 1 < n, kv && j0 + 2 < n, kv && j0 + 3 < n, v);
#pragma unroll
                for (int j = 0; j < DT; ++j) b[kk][j] = v[j];
            }
        }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)      // increasing k: every entry of C is one dot product summed in order
#pragma unroll
            for (int j = 0; j < DT; ++j)
#pragma unroll
                for (int i = 0; i < DT; ++i) acc[j][i] = fmaf(a[kk][i], b[kk][j], acc[j][i]);
    }

    // alpha / beta of Fig. 3 at the store; C is not read when beta == 0
    const bool cvec = VEC && rows_in && ldc % 4 == 0 && strideC % 4 == 0 && (reinterpret_cast<uintptr_t>(C) & 15) == 0;
#pragma unroll
    for (int j = 0; j < DT; ++j) {
        if (j0 + j >= n) break;
        float* c = C + i0 + (j0 + j) * ldc;
        if (cvec) {
            float4 r = make_float4(alpha * acc[j][0], alpha * acc[j][1], alpha * acc[j][2], alpha * acc[j][3]);
            if (beta != 0.0f) {
                const float4 c0 = *reinterpret_cast<const float4*>(c);
                r.x = fmaf(beta, c0.x, r.x); r.y = fmaf(beta, c0.y, r.y);
                r.z = fmaf(beta, c0.z, r.z); r.w = fmaf(beta, c0.w, r.w);
            }
            *reinterpret_cast<float4*>(c) = r;
        } else {
#pragma unroll
            for (int i = 0; i < DT; ++i)
                if (i0 + i < m) {
                    float r = alpha * acc[j][i];
                    if (beta != 0.0f) r = fmaf(beta, c[i], r);
                    c[i] = r;
                }
        }
    }
}

template <bool TA, bool TB, bool VEC>
static cudaError_t launch_direct_t(const GemmArgs& a, int64_t sA, int64_t sB, int64_t sC, int64_t tiles_m, int64_t spp,
                                   int64_t total) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)((total + D_WARPS - 1) / D_WARPS), 1, 1);
    lc.blockDim = dim3(32 * D_WARPS);
    lc.stream = a.stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // pairs with griddepcontrol.wait in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    cudaError_t le = cudaLaunchKernelEx(&lc, simt_direct_kernel<TA, TB, VEC>, a.m, a.n, a.k, a.alpha, (const float*)a.A, a.lda, sA,
                                        (const float*)a.B, a.ldb, sB, a.beta, a.C, a.ldc, sC, (int)tiles_m, spp, total);
    return le != cudaSuccess ? le : cudaGetLastError();
}

cudaError_t launch_simt_direct(const GemmArgs& a, int64_t strideA, int64_t strideB, int64_t strideC, int64_t batch,
                               gemm_config_t* cfg) {
    const int64_t tiles_m = (a.m + D_TILE_M - 1) / D_TILE_M, tiles_n = (a.n + D_TILE_N - 1) / D_TILE_N;
    const int64_t spp = tiles_m * tiles_n;                    // slabs per problem
    if (batch < 1 || tiles_m > 0x7FFFFFFF || spp > (1LL << 40) / batch) return cudaErrorInvalidConfiguration;
    const int64_t total = spp * batch;
    if ((total + D_WARPS - 1) / D_WARPS > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    auto al = [](const void* p, int64_t ld, int64_t stride) {
        return (reinterpret_cast<uintptr_t>(p) & 15) == 0 && ld % 4 == 0 && stride % 4 == 0;
    };
    const bool vec = al(a.A, a.lda, strideA) && al(a.B, a.ldb, strideB);
    cfg->kernel = GEMM_KERNEL_SIMT_DIRECT;
    cfg->tile_m = D_TILE_M; cfg->tile_n = D_TILE_N; cfg->tile_k = 4; cfg->split_k = 1; cfg->stages = 1;
    const int64_t ctas = (total + D_WARPS - 1) / D_WARPS;
    cfg->grid = (int32_t)(ctas > 0x7FFFFFFF ? 0x7FFFFFFF : ctas);
    cfg->vector_a = cfg->vector_b = vec ? 4 : 1;
    cfg->launches = 1;
#define DIRECT(TA_, TB_) (vec ? launch_direct_t<TA_, TB_, true>(a, strideA, strideB, strideC, tiles_m, spp, total) \
                              : launch_direct_t<TA_, TB_, false>(a, strideA, strideB, strideC, tiles_m, spp, total))
    if (!a.ta && !a.tb) return DIRECT(false, false);
    if (a.ta && !a.tb) return DIRECT(true, false);
    if (!a.ta && a.tb) return DIRECT(false, true);
    return DIRECT(true, true);
#undef DIRECT
}

}  // namespace b200gemm
