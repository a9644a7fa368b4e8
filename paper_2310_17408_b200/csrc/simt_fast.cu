// Fast fp32 GEMM on the CUDA cores (exact IEEE fp32 FMA).
//
// Mapping of the paper's algorithm (Fig. 1) onto the SM:
//   loops L1/L3 (jc, ic)   -> grid of BM x BN CTA tiles of C, visited in groups of tile rows so that the CTAs
//                             resident at one time share their A and B panels in L2
//   loop  L2 (pc, kc)      -> the CTA's loop over BK = 16 slices of k (optionally a k range per CTA: split-k)
//   Pack-A / Pack-B        -> 128-bit global loads into registers, stored to a double-buffered shared-memory
//                             stage laid out [k][m] and [k][n] so that a thread's fragment is one 128-bit read
//   loops L4/L5 + L6       -> each warp owns a 64 x 32 sub-tile, each thread an 8 x 8 register block that
//                             receives one outer product per k (the role of the mr x nr micro-kernel)
//   alpha / beta (Fig. 3)  -> applied once, when the register block is stored
#include <atomic>

#include "internal.cuh"

namespace b200gemm {

constexpr int BK = 16;
constexpr int PAD = 4;   // row padding of the shared-memory stage (floats); keeps rows 16-byte aligned

// ---- global -> register loader for one operand tile of X_TILE (m or n extent) x BK
// KCONT: the stored matrix is contiguous along k (A with transA = T, B with transB = N);
// otherwise it is contiguous along the tile dimension.  VEC: elements per load (4 needs 16-byte alignment).
template <int X_TILE, int NT, bool KCONT, int VEC>
struct Loader {
    static constexpr int ELEMS = X_TILE * BK / NT;   // per thread
    static constexpr int NV = ELEMS / VEC;           // loads per thread
    static_assert(ELEMS % VEC == 0 && ELEMS >= VEC, "tile / thread count mismatch");

    // coordinates (x, kk) of load v of thread t; a VEC=4 load covers 4 consecutive elements of the contiguous dim
    __device__ static __forceinline__ void coord(int t, int v, int& x, int& kk) {
        if (KCONT) {
            constexpr int KV = BK / VEC;             // loads along k per row
            kk = (t % KV) * VEC;
            x = t / KV + v * (NT / KV);
        } else {
            constexpr int XV = X_TILE / VEC;
            x = (t % XV) * VEC;
            kk = t / XV + v * (NT / XV);
        }
    }

    template <bool GUARD>
    __device__ static __forceinline__ void load(float (&r)[ELEMS], const float* __restrict__ X, int64_t ld,
                                                int64_t x0, int64_t k0, int64_t xmax, int64_t kmax, int t) {
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            int x, kk;
            coord(t, v, x, kk);
            int64_t gx = x0 + x, gk = k0 + kk;
            const float* p = KCONT ? X + gk + gx * ld : X + gx + gk * ld;
            if (VEC == 4) {
                bool whole = !GUARD || (KCONT ? (gx < xmax && gk + 3 < kmax) : (gx + 3 < xmax && gk < kmax));
                if (whole) {
                    float4 q = __ldg(reinterpret_cast<const float4*>(p));
                    r[v * 4 + 0] = q.x; r[v * 4 + 1] = q.y; r[v * 4 + 2] = q.z; r[v * 4 + 3] = q.w;
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        bool ok = KCONT ? (gx < xmax && gk + c < kmax) : (gx + c < xmax && gk < kmax);
                        r[v * 4 + c] = ok ? __ldg(p + c) : 0.0f;
                    }
                }
            } else {
                bool ok = !GUARD || (gx < xmax && gk < kmax);
                r[v] = ok ? __ldg(p) : 0.0f;
            }
        }
    }

    // Unguarded loads through a running pointer: `p0` addresses load 0 of this thread in the current k slice,
    // `vstride` is the element distance between consecutive loads of the thread (fixed for the whole call).
    __device__ static __forceinline__ int64_t load_stride(int64_t ld) {
        return KCONT ? (int64_t)(NT / (BK / VEC)) * ld : (int64_t)(NT / (X_TILE / VEC)) * ld;
    }
    __device__ static __forceinline__ const float* first_load(const float* X, int64_t ld, int64_t x0, int64_t k0, int t) {
        int x, kk;
        coord(t, 0, x, kk);
        return KCONT ? X + (k0 + kk) + (x0 + x) * ld : X + (x0 + x) + (k0 + kk) * ld;
    }
    __device__ static __forceinline__ void load_fast(float (&r)[ELEMS], const float* __restrict__ p0, int64_t vstride) {
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const float* p = p0 + v * vstride;
            if (VEC == 4) {
                float4 q = __ldg(reinterpret_cast<const float4*>(p));
                r[v * 4 + 0] = q.x; r[v * 4 + 1] = q.y; r[v * 4 + 2] = q.z; r[v * 4 + 3] = q.w;
            } else {
                r[v] = __ldg(p);
            }
        }
    }

    // registers -> shared stage S[kk][x] (row length X_TILE + PAD)
    __device__ static __forceinline__ void store(const float (&r)[ELEMS], float* S, int t) {
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            int x, kk;
            coord(t, v, x, kk);
            if (VEC == 4) {
                if (KCONT) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) S[(kk + c) * (X_TILE + PAD) + x] = r[v * 4 + c];
                } else {
                    *reinterpret_cast<float4*>(S + kk * (X_TILE + PAD) + x) =
                        make_float4(r[v * 4 + 0], r[v * 4 + 1], r[v * 4 + 2], r[v * 4 + 3]);
                }
            } else {
                S[kk * (X_TILE + PAD) + x] = r[v];
            }
        }
    }
};

// ---- operand B read through the im2row index map (the lowering fused into Pack-B): the tile's BN columns are
// output pixels, its k index runs over (r, s, c).  Register layout and shared-memory store are those of the
// k-contiguous Loader, so the rest of the kernel does not change.  VEC = 4 needs C_in % 4 == 0 and a 16-byte
// aligned tensor: four consecutive k are then four consecutive channels of one filter tap.
template <int X_TILE, int NT, int VEC>
struct ConvLoader {
    using L = Loader<X_TILE, NT, true, VEC>;
    static constexpr int ELEMS = L::ELEMS, NV = L::NV;

    // per load of the thread: element offset of pixel (b, ho*sh - ph, wo*sw - pw) and those two coordinates;
    // a column past the last pixel gets coordinates that fail every bounds check
    struct Pixel {
        int64_t off;
        int h0, w0;
    };
    __device__ static __forceinline__ Pixel pixel(const ConvIndex& cv, int64_t j, int64_t n) {
        Pixel px;
        if (j >= n) { px.off = 0; px.h0 = px.w0 = -(1 << 29); return px; }
        const int hw = cv.ho * cv.wo;
        const int b = (int)(j / hw), rem = (int)(j - (int64_t)b * hw);
        const int oh = rem / cv.wo, ow = rem - oh * cv.wo;
        px.h0 = oh * cv.sh - cv.ph;
        px.w0 = ow * cv.sw - cv.pw;
        px.off = (((int64_t)b * cv.h + px.h0) * cv.w + px.w0) * cv.c_in;
        return px;
    }

    // Position of the thread's k index inside the filter: tap (fr, fs) and channel c.  All loads of a thread share
    // it (their kk is the same), and it moves forward by one k slice per load() call, so it is kept as running
    // state instead of being divided out of p every time.
    struct Tap {
        int fr, fs, c;
        int64_t p;
    };
    __device__ static __forceinline__ Tap first_tap(const ConvIndex& cv, int64_t kbeg, int t) {
        int x, kk;
        L::coord(t, 0, x, kk);
        Tap tp;
        tp.p = kbeg + kk;
        const uint32_t p32 = (uint32_t)tp.p, cin = (uint32_t)cv.c_in;       // k = kh*kw*C_in fits 31 bits (checked by the host)
        const uint32_t tap = p32 / cin;
        tp.c = (int)(p32 - tap * cin);
        tp.fr = (int)(tap / (uint32_t)cv.kw);
        tp.fs = (int)(tap - (uint32_t)tp.fr * (uint32_t)cv.kw);
        return tp;
    }
    __device__ static __forceinline__ void advance(const ConvIndex& cv, Tap& tp) {
        tp.p += BK;
        tp.c += BK;
        const int cin = (int)cv.c_in;
        while (tp.c >= cin) {
            tp.c -= cin;
            if (++tp.fs == cv.kw) { tp.fs = 0; ++tp.fr; }
        }
    }

    __device__ static __forceinline__ void load(float (&r)[ELEMS], const ConvIndex& cv, const Pixel (&px)[VEC == 4 ? NV : 1],
                                                Tap& tp, int64_t j0, int64_t n, int64_t kmax, int t) {
        const float* __restrict__ X = static_cast<const float*>(cv.X);
        const bool k_ok = tp.p < kmax;            // VEC = 4: k is a multiple of 4 here, so the four elements share it
        const int64_t tap_off = ((int64_t)tp.fr * cv.w + tp.fs) * cv.c_in + tp.c;
        const int fr = tp.fr, fs = tp.fs;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            if (VEC == 4) {
                const int hi = px[v].h0 + fr, wi = px[v].w0 + fs;
                float4 q = make_float4(0.f, 0.f, 0.f, 0.f);
                if (k_ok && (unsigned)hi < (unsigned)cv.h && (unsigned)wi < (unsigned)cv.w)
                    q = __ldg(reinterpret_cast<const float4*>(X + px[v].off + tap_off));
                r[v * 4 + 0] = q.x; r[v * 4 + 1] = q.y; r[v * 4 + 2] = q.z; r[v * 4 + 3] = q.w;
            } else {
                int x, kk;
                L::coord(t, v, x, kk);
                const Pixel one = pixel(cv, j0 + x, n);
                const int hi = one.h0 + fr, wi = one.w0 + fs;
                r[v] = (k_ok && (unsigned)hi < (unsigned)cv.h && (unsigned)wi < (unsigned)cv.w) ? __ldg(X + one.off + tap_off) : 0.0f;
            }
        }
        advance(cv, tp);
    }
};

// Packed fp32 arithmetic: one fma.rn.f32x2 performs two independent IEEE fp32 fused multiply-adds (round to nearest
// even, no flush to zero), lo = a.lo*b.lo + c.lo and hi = a.hi*b.hi + c.hi, in one issue slot.  It halves the
// instructions of the products (issue slots used: 83 % -> 49 %); the FMA pipes themselves then set the pace.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma2(uint64_t& c, uint64_t a, uint64_t b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(c) : "l"(a), "l"(b));
}

// The thread's 8 x 8 register block as packed pairs of neighbouring columns: P[i][j] = ( acc(i, 2j), acc(i, 2j+1) ),
// updated with (a_i, a_i) * (b_2j, b_2j+1).  The pairs of B come straight out of the 128-bit fragment loads; every a_i
// is duplicated into a pair once per k; column pair by column pair, so that eight consecutive instructions share the
// B pair.  Forms measured in this kernel at 8192^3: this one 59.7 TFLOP/s; pairs of neighbouring rows with b
// duplicated 58.1 (either order of the loops); pairs along the diagonals (A pairs and swapped B pairs, no duplicates)
// 55.3; the scalar block 51 (at 4096^3).  On operands fed from shared memory alone, without the global loads, stores and barriers
// around it, the same forms reach 66, 63-66, 61 and 60-63.
struct Acc2 {
    uint64_t P[8][4];
};

// one BK slice of outer products on the thread's 8 x 8 register block
template <int BM, int BN>
__device__ __forceinline__ void compute_stage(Acc2& acc, const float* __restrict__ As,
                                              const float* __restrict__ Bs, int am, int bn) {
    uint64_t a[2][8], b[2][4];
    auto frag = [&](int kk, int buf) {
        const float* ap = As + kk * (BM + PAD) + am;
        const float* bp = Bs + kk * (BN + PAD) + bn;
        float4 a0 = *reinterpret_cast<const float4*>(ap);
        float4 a1 = *reinterpret_cast<const float4*>(ap + 32);
        float4 b0 = *reinterpret_cast<const float4*>(bp);
        float4 b1 = *reinterpret_cast<const float4*>(bp + 16);
        b[buf][0] = pack2(b0.x, b0.y); b[buf][1] = pack2(b0.z, b0.w);
        b[buf][2] = pack2(b1.x, b1.y); b[buf][3] = pack2(b1.z, b1.w);
        a[buf][0] = pack2(a0.x, a0.x); a[buf][1] = pack2(a0.y, a0.y);
        a[buf][2] = pack2(a0.z, a0.z); a[buf][3] = pack2(a0.w, a0.w);
        a[buf][4] = pack2(a1.x, a1.x); a[buf][5] = pack2(a1.y, a1.y);
        a[buf][6] = pack2(a1.z, a1.z); a[buf][7] = pack2(a1.w, a1.w);
    };
    frag(0, 0);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
        if (kk + 1 < BK) frag(kk + 1, (kk + 1) & 1);
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int i = 0; i < 8; ++i) fma2(acc.P[i][j], a[kk & 1][i], b[kk & 1][j]);
    }
}

// packed accumulators -> acc[column][row] of the 8 x 8 block
__device__ __forceinline__ void unpack_block(const Acc2& p, float (&acc)[8][8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) unpack2(p.P[i][j], acc[2 * j][i], acc[2 * j + 1][i]);
}

// Whether the kernel with this CTA tile can finish a split of k itself, as a thread-block cluster: every CTA then
// parks its BM x BN partial sums in shared memory, which the operand stages are reused for (64 KB for 128 x 128:
// more than a statically allocated array may have, so that tile keeps the workspace and the reduction pass).
template <int BM, int BN> struct ClusterReduce { static constexpr bool value = !(BM == 128 && BN == 128); };

__device__ __forceinline__ uint32_t map_shared_to_cta(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 ld_cluster_f4(uint32_t cluster_addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr));
    return v;
}
__device__ __forceinline__ void cluster_barrier() {      // all threads of all CTAs of the cluster
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int BM, int BN, int WARPS_M, int WARPS_N, int MINB, bool A_KCONT, bool B_KCONT, int VA, int VB, bool CONV>
__device__ __forceinline__ void
simt_fast_body(int64_t m, int64_t n, int64_t k, float alpha, const float* __restrict__ A, int64_t lda,
               const float* __restrict__ B, int64_t ldb, float beta, float* __restrict__ C, int64_t ldc,
               int tiles_m, int tiles_n, int64_t kchunk, float* __restrict__ partials, const SimtExtra& ex,
               const ConvIndex& cv) {
    const TailSplit& tail = ex.tail;

    constexpr int NT = WARPS_M * WARPS_N * 32;
    static_assert(BM == WARPS_M * 64 && BN == WARPS_N * 32, "warp tile is 64 x 32");
    using LA = Loader<BM, NT, A_KCONT, VA>;
    using LB = Loader<BN, NT, B_KCONT, VB>;
    using LC = ConvLoader<BN, NT, VB>;

    constexpr int A_STAGE = BK * (BM + PAD), B_STAGE = BK * (BN + PAD);
    constexpr int STAGE_FLOATS = 2 * A_STAGE + 2 * B_STAGE;
    constexpr int SMEM_FLOATS = (ClusterReduce<BM, BN>::value && BM * BN > STAGE_FLOATS) ? BM * BN : STAGE_FLOATS;
    __shared__ __align__(16) float smem[SMEM_FLOATS];      // operand stages; at the end the tile's partial sums (cluster reduction)
    float (*As)[A_STAGE] = reinterpret_cast<float (*)[A_STAGE]>(smem);
    float (*Bs)[B_STAGE] = reinterpret_cast<float (*)[B_STAGE]>(smem + 2 * A_STAGE);

    // programmatic dependent launch: the next kernel of the stream may be scheduled once every CTA of this one
    // has started; it waits (griddepcontrol.wait) before it touches global memory, as this kernel does below
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int t = threadIdx.x;
    const int warp = t >> 5, lane = t & 31;
    const int wm = warp % WARPS_M, wn = warp / WARPS_M;
    const int lm = lane & 7, ln = lane >> 3;          // 8 lanes along m, 4 along n
    const int am = wm * 64 + lm * 4;                  // thread rows: am..am+3 and am+32..am+35
    const int bn = wn * 32 + ln * 4;                  // thread cols: bn..bn+3 and bn+16..bn+19

    // Work items: blockIdx.x < tail.first is one whole tile.  The tiles of the last, partly filled wave
    // (tail.first and up) are cut into tail.splits k ranges each, so that the wave still fills the machine;
    // their raw partial sums go to tile-local slots of tail.partials and a small reduction pass finishes them.
    int tile = blockIdx.x, ksplit = blockIdx.z;
    int64_t kc = kchunk;
    float* tail_out = nullptr;
    if (tile >= tail.first) {
        const int item = tile - tail.first;
        tile = tail.first + item / tail.splits;
        ksplit = item % tail.splits;
        kc = tail.chunk;
        tail_out = tail.partials + (int64_t)item * (BM * BN);
    }
    int tm, tn;
    decode_tile(tile, tiles_m, tiles_n, &tm, &tn);
    const int64_t i0 = (int64_t)tm * BM, j0 = (int64_t)tn * BN;

    const int64_t kbeg = (int64_t)ksplit * kc;
    const int64_t kend = min(k, kbeg + kc);
    const int64_t ktiles = (kend - kbeg + BK - 1) / BK;

    Acc2 acc2;
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc2.P[j][i] = 0ull;      // (+0.0f, +0.0f)

    float ra[LA::ELEMS], rb[LB::ELEMS];
    const bool interior = (i0 + BM <= m) && (j0 + BN <= n);

    // interior tiles read whole k slices through running pointers; edge tiles and the k tail take the guarded path
    const float* pa = LA::first_load(A, lda, i0, kbeg, t);
    const float* pb = LB::first_load(B, ldb, j0, kbeg, t);
    const int64_t va = LA::load_stride(lda), vb = LB::load_stride(ldb);
    const int64_t step_a = A_KCONT ? (int64_t)BK : (int64_t)BK * lda;
    const int64_t step_b = B_KCONT ? (int64_t)BK : (int64_t)BK * ldb;
    const int64_t fast_tiles = interior ? (kend - kbeg) / BK : 0;

    // im2row index map: the pixels of this thread's loads are fixed for the whole k loop
    typename LC::Pixel px[VB == 4 ? LC::NV : 1];
    if (CONV && VB == 4) {
#pragma unroll
        for (int v = 0; v < LC::NV; ++v) {
            int x, kk;
            LB::coord(t, v, x, kk);
            px[v] = LC::pixel(cv, j0 + x, n);
        }
    }

    typename LC::Tap tap{0, 0, 0, 0};
    if (CONV) tap = LC::first_tap(cv, kbeg, t);

    auto gload = [&](int64_t kt) {      // called for kt = 0, 1, 2, ... in order
        if (kt < fast_tiles) {
            LA::load_fast(ra, pa, va);
            pa += step_a;
            if (!CONV) {
                LB::load_fast(rb, pb, vb);
                pb += step_b;
            }
        } else {
            const int64_t k0 = kbeg + kt * BK;
            LA::template load<true>(ra, A, lda, i0, k0, m, kend, t);
            if (!CONV) LB::template load<true>(rb, B, ldb, j0, k0, n, kend, t);
        }
        if (CONV) LC::load(rb, cv, px, tap, j0, n, kend, t);
    };

    asm volatile("griddepcontrol.wait;" ::: "memory");     // the previous kernel's results are visible from here on
    if (ktiles > 0) {
        gload(0);
        LA::store(ra, As[0], t);
        LB::store(rb, Bs[0], t);
        __syncthreads();
        for (int64_t kt = 0; kt < ktiles; ++kt) {
            const int cur = (int)(kt & 1);
            if (kt + 1 < ktiles) gload(kt + 1);                 // in flight during the math below
            compute_stage<BM, BN>(acc2, As[cur], Bs[cur], am, bn);
            if (kt + 1 < ktiles) {
                LA::store(ra, As[cur ^ 1], t);
                LB::store(rb, Bs[cur ^ 1], t);
            }
            __syncthreads();
        }
    }

    // ---- store: alpha*acc + beta*C, or raw partial sums for split-k
    float acc[8][8];
    unpack_block(acc2, acc);
    if (tail_out != nullptr) {      // tile-local slot [BN][BM]: whole register blocks, no bounds (edge entries are zero)
#pragma unroll
        for (int jh = 0; jh < 2; ++jh)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj)
#pragma unroll
                for (int ih = 0; ih < 2; ++ih) {
                    const float* v = &acc[jh * 4 + jj][ih * 4];
                    *reinterpret_cast<float4*>(tail_out + (am + ih * 32) + (bn + jh * 16 + jj) * BM) =
                        make_float4(v[0], v[1], v[2], v[3]);
                }
        return;
    }
    if constexpr (ClusterReduce<BM, BN>::value) {
        if (ex.cluster_reduce) {
            // Split k finished by the cluster that holds this tile's k ranges (cluster rank = split index = blockIdx.z).
            // Park the register block in shared memory as a dense [BN][BM] tile, ...
            const int splits = (int)gridDim.z, rank = (int)blockIdx.z;
#pragma unroll
            for (int jh = 0; jh < 2; ++jh)
#pragma unroll
                for (int jj = 0; jj < 4; ++jj)
#pragma unroll
                    for (int ih = 0; ih < 2; ++ih) {
                        const float* v = &acc[jh * 4 + jj][ih * 4];
                        *reinterpret_cast<float4*>(smem + (am + ih * 32) + (bn + jh * 16 + jj) * BM) = make_float4(v[0], v[1], v[2], v[3]);
                    }
            cluster_barrier();
            // ... then this CTA sums its share of the tile (a contiguous run of its columns) over all CTAs, in
            // increasing split index whoever does the summing, reading the others' shared memory
            const bool cvec = ((reinterpret_cast<uintptr_t>(C) & 15) == 0) && (ldc % 4 == 0);
            const uint32_t base = (uint32_t)__cvta_generic_to_shared(smem);
            constexpr int VECS = BM * BN / 4;
            const int share = (VECS + splits - 1) / splits;
            const int v_end = min(VECS, (rank + 1) * share);
            for (int v4 = rank * share + t; v4 < v_end; v4 += NT) {
                const int e = v4 * 4, r = e % BM, c = e / BM;
                float4 q[CLUSTER_REDUCE_MAX_SPLITS];
#pragma unroll
                for (int z = 0; z < CLUSTER_REDUCE_MAX_SPLITS; ++z)
                    if (z < splits) q[z] = ld_cluster_f4(map_shared_to_cta(base + (uint32_t)e * 4u, (uint32_t)z));
                float4 s4 = q[0];
#pragma unroll
                for (int z = 1; z < CLUSTER_REDUCE_MAX_SPLITS; ++z)
                    if (z < splits) { s4.x += q[z].x; s4.y += q[z].y; s4.z += q[z].z; s4.w += q[z].w; }
                const int64_t gi = i0 + r, gj = j0 + c;
                if (gi >= m || gj >= n) continue;
                float* cp = C + gi + gj * ldc;
                if (cvec && gi + 3 < m) {
                    float4 o = make_float4(alpha * s4.x, alpha * s4.y, alpha * s4.z, alpha * s4.w);
                    if (beta != 0.0f) {
                        const float4 c0 = *reinterpret_cast<const float4*>(cp);
                        o.x = fmaf(beta, c0.x, o.x); o.y = fmaf(beta, c0.y, o.y);
                        o.z = fmaf(beta, c0.z, o.z); o.w = fmaf(beta, c0.w, o.w);
                    }
                    *reinterpret_cast<float4*>(cp) = o;
                } else {
                    const float sv[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4)
                        if (gi + q4 < m) {
                            float o = alpha * sv[q4];
                            if (beta != 0.0f) o = fmaf(beta, cp[q4], o);
                            cp[q4] = o;
                        }
                }
            }
            cluster_barrier();      // nobody leaves while its shared memory may still be read
            return;
        }
    }
    const bool raw = partials != nullptr;
    float* out = raw ? partials + (int64_t)blockIdx.z * m * n : C;
    const int64_t ldo = raw ? m : ldc;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(out) & 15) == 0) && (ldo % 4 == 0);
#pragma unroll
    for (int jh = 0; jh < 2; ++jh)
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const int64_t gj = j0 + bn + jh * 16 + jj;
            if (gj >= n) continue;
#pragma unroll
            for (int ih = 0; ih < 2; ++ih) {
                const int64_t gi = i0 + am + ih * 32;
                float* c = out + gi + gj * ldo;
                const float* v = &acc[jh * 4 + jj][ih * 4];
                if (vec_ok && gi + 3 < m) {
                    float4 r;
                    if (raw) {
                        r = make_float4(v[0], v[1], v[2], v[3]);
                    } else {
                        r = make_float4(alpha * v[0], alpha * v[1], alpha * v[2], alpha * v[3]);
                        if (beta != 0.0f) {
                            float4 c0 = *reinterpret_cast<const float4*>(c);
                            r.x = fmaf(beta, c0.x, r.x); r.y = fmaf(beta, c0.y, r.y);
                            r.z = fmaf(beta, c0.z, r.z); r.w = fmaf(beta, c0.w, r.w);
                        }
                    }
                    *reinterpret_cast<float4*>(c) = r;
                } else {
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        if (gi + e < m) {
                            float r = raw ? v[e] : alpha * v[e];
                            if (!raw && beta != 0.0f) r = fmaf(beta, c[e], r);
                            c[e] = r;
                        }
                }
            }
        }

}

template <int BM, int BN, int WARPS_M, int WARPS_N, int MINB, bool A_KCONT, bool B_KCONT, int VA, int VB>
__global__ void __launch_bounds__(WARPS_M* WARPS_N * 32, MINB)
simt_fast_kernel(int64_t m, int64_t n, int64_t k, float alpha, const float* __restrict__ A, int64_t lda,
                 const float* __restrict__ B, int64_t ldb, float beta, float* __restrict__ C, int64_t ldc,
                 int tiles_m, int tiles_n, int64_t kchunk, float* __restrict__ partials, SimtExtra ex) {
    simt_fast_body<BM, BN, WARPS_M, WARPS_N, MINB, A_KCONT, B_KCONT, VA, VB, false>(
        m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, tiles_m, tiles_n, kchunk, partials, ex, ConvIndex{});
}

// a strided batch of problems of one shape: blockIdx.y is the problem (instantiated for the 64 x 64 and 128 x 128 CTA
// tiles; a kernel of its own, because the three extra pointer offsets cost the single-problem kernel registers it
// does not have)
template <int BM, int BN, int WARPS_M, int WARPS_N, int MINB, bool A_KCONT, bool B_KCONT, int VA, int VB>
__global__ void __launch_bounds__(WARPS_M* WARPS_N * 32, MINB)
simt_batched_kernel(int64_t m, int64_t n, int64_t k, float alpha, const float* __restrict__ A, int64_t lda,
                    const float* __restrict__ B, int64_t ldb, float beta, float* __restrict__ C, int64_t ldc,
                    int tiles_m, int tiles_n, int64_t kchunk, SimtExtra ex) {
    simt_fast_body<BM, BN, WARPS_M, WARPS_N, MINB, A_KCONT, B_KCONT, VA, VB, false>(
        m, n, k, alpha, A + (int64_t)blockIdx.y * ex.strideA, lda, B + (int64_t)blockIdx.y * ex.strideB, ldb, beta,
        C + (int64_t)blockIdx.y * ex.strideC, ldc, tiles_m, tiles_n, kchunk, nullptr, ex, ConvIndex{});
}

// the same kernel with operand B read through the im2row index map (n = output pixels, k = kh*kw*C_in)
template <int BM, int BN, int WARPS_M, int WARPS_N, int MINB, bool A_KCONT, int VA, int VB>
__global__ void __launch_bounds__(WARPS_M* WARPS_N * 32, MINB)
simt_conv_kernel(int64_t m, int64_t n, int64_t k, float alpha, const float* __restrict__ A, int64_t lda,
                 float beta, float* __restrict__ C, int64_t ldc, int tiles_m, int tiles_n, int64_t kchunk,
                 float* __restrict__ partials, SimtExtra ex, const ConvIndex cv) {
    simt_fast_body<BM, BN, WARPS_M, WARPS_N, MINB, A_KCONT, true, VA, VB, true>(
        m, n, k, alpha, A, lda, nullptr, k, beta, C, ldc, tiles_m, tiles_n, kchunk, partials, ex, cv);
}

// ---------------------------------------------------------------- host side

bool simt_fast_can_cluster_reduce(int tile) { return tile != 0; }      // see ClusterReduce

bool simt_fast_eligible(const GemmArgs& a, int* va, int* vb) {
    if (a.dtype != GEMM_F32) return false;
    auto vec = [](const void* p, int64_t ld) { return ((reinterpret_cast<uintptr_t>(p) & 15) == 0 && ld % 4 == 0) ? 4 : 1; };
    *va = vec(a.A, a.lda);
    *vb = vec(a.B, a.ldb);
    return true;
}

template <int BM, int BN, int WM, int WN, int MINB, bool AK, bool BKC, int VA, int VB>
static cudaError_t launch_one(const GemmArgs& a, KSplit ks, float* partials, gemm_config_t* cfg, const SimtExtra& ex, int64_t batch) {
    const TailSplit& tail = ex.tail;
    int64_t tiles_m = (a.m + BM - 1) / BM, tiles_n = (a.n + BN - 1) / BN;
    if (tiles_m * tiles_n > 0x7FFFFFFFLL || tiles_m > 0x7FFFFFFF || tiles_n > 0x7FFFFFFF / 16)
        return cudaErrorInvalidConfiguration;       // tile indices are 32-bit in the kernel (groups of 16 tile rows)
    int64_t items = tiles_m * tiles_n;
    if (tail.first < items) items = tail.first + (items - tail.first) * tail.splits;      // tail tiles count once per k range
    if (items > 0x7FFFFFFFLL || batch < 1 || batch > 65535) return cudaErrorInvalidConfiguration;
    dim3 grid((unsigned)items, (unsigned)batch, (unsigned)ks.splits);
    cfg->tile_m = BM; cfg->tile_n = BN; cfg->tile_k = BK; cfg->stages = 2;
    const int64_t ctas = items * ks.splits * batch;
    cfg->grid = (int32_t)(ctas > 0x7FFFFFFF ? 0x7FFFFFFF : ctas);
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid;
    lc.blockDim = dim3(WM * WN * 32);
    lc.stream = a.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // pairs with griddepcontrol.wait in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (ex.cluster_reduce) {      // the k ranges of one tile form a cluster along z
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = 1;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = (unsigned)ks.splits;
        lc.numAttrs = 2;
        // The CTAs of a cluster are placed close together, several to an SM where they fit, which leaves SMs idle
        // when the whole grid is small.  Unused dynamic shared memory is requested so that no more CTAs fit on an
        // SM than an even spread over all SMs needs (a cluster launch is split-k: always a small grid).
        if constexpr (!BKC || true) {
            auto kern = simt_fast_kernel<BM, BN, WM, WN, MINB, AK, BKC, VA, VB>;
            static std::atomic<int> static_smem[64];      // per device: static shared memory of this kernel, 0 = not asked yet
            int dev = 0;
            cudaGetDevice(&dev);
            const int sms = sm_count();
            int per_sm = (int)((ctas + sms - 1) / sms);
            if (dev >= 0 && dev < 64 && per_sm < MINB && a.conv == nullptr) {
                int st = static_smem[dev].load();
                if (st == 0) {
                    cudaFuncAttributes fa;
                    if (cudaFuncGetAttributes(&fa, kern) == cudaSuccess &&
                        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 190 * 1024) == cudaSuccess) {
                        st = (int)fa.sharedSizeBytes + 1024;      // + what the system reserves per CTA
                        static_smem[dev].store(st);
                    } else {
                        (void)cudaGetLastError();
                    }
                }
                if (st > 0) {
                    const int total = 228 * 1024 / (per_sm + 1) + 2048;      // per CTA: per_sm fit on an SM, per_sm + 1 do not
                    if (total > st && total * per_sm <= 228 * 1024) lc.dynamicSmemBytes = (size_t)(total - st);
                }
            }
        }
    }
    cudaError_t le;
    if constexpr (BKC) {
        if (a.conv != nullptr) {      // operand B through the im2row index map (its memory layout is k-contiguous by construction)
            le = cudaLaunchKernelEx(&lc, simt_conv_kernel<BM, BN, WM, WN, MINB, AK, VA, VB>, a.m, a.n, a.k, a.alpha,
                                    (const float*)a.A, a.lda, a.beta, a.C, a.ldc, (int)tiles_m, (int)tiles_n, ks.chunk,
                                    ks.splits > 1 ? partials : (float*)nullptr, ex, *a.conv);
            return le != cudaSuccess ? le : cudaGetLastError();
        }
    }
    if (batch > 1 || ex.strideA != 0 || ex.strideB != 0 || ex.strideC != 0) {
        if constexpr ((BM == 64 && BN == 64) || (BM == 128 && BN == 128)) {
            le = cudaLaunchKernelEx(&lc, simt_batched_kernel<BM, BN, WM, WN, MINB, AK, BKC, VA, VB>, a.m, a.n, a.k, a.alpha,
                                    (const float*)a.A, a.lda, (const float*)a.B, a.ldb, a.beta, a.C, a.ldc,
                                    (int)tiles_m, (int)tiles_n, ks.chunk, ex);
            return le != cudaSuccess ? le : cudaGetLastError();
        } else {
            return cudaErrorInvalidConfiguration;      // batches run on the 64 x 64 and 128 x 128 tiles only
        }
    }
    le = cudaLaunchKernelEx(&lc, simt_fast_kernel<BM, BN, WM, WN, MINB, AK, BKC, VA, VB>, a.m, a.n, a.k, a.alpha,
                            (const float*)a.A, a.lda, (const float*)a.B, a.ldb, a.beta, a.C, a.ldc,
                            (int)tiles_m, (int)tiles_n, ks.chunk,
                            ks.splits > 1 ? partials : (float*)nullptr, ex);
    return le != cudaSuccess ? le : cudaGetLastError();
}

template <bool AK, bool BKC, int VA, int VB>
static cudaError_t launch_tile(const GemmArgs& a, int tile, KSplit ks, float* partials, gemm_config_t* cfg, const SimtExtra& ex, int64_t batch) {
    switch (tile) {
        case 0: return launch_one<128, 128, 2, 4, 2, AK, BKC, VA, VB>(a, ks, partials, cfg, ex, batch);
        case 1: return launch_one<128, 64, 2, 2, 3, AK, BKC, VA, VB>(a, ks, partials, cfg, ex, batch);
        case 2: return launch_one<64, 128, 1, 4, 3, AK, BKC, VA, VB>(a, ks, partials, cfg, ex, batch);
        default: return launch_one<64, 64, 1, 2, 6, AK, BKC, VA, VB>(a, ks, partials, cfg, ex, batch);
    }
}

template <bool AK, bool BKC>
static cudaError_t launch_vec(const GemmArgs& a, int va, int vb, int tile, KSplit ks, float* partials,
                              gemm_config_t* cfg, const SimtExtra& ex, int64_t batch) {
    if (va == 4 && vb == 4) return launch_tile<AK, BKC, 4, 4>(a, tile, ks, partials, cfg, ex, batch);
    if (va == 4) return launch_tile<AK, BKC, 4, 1>(a, tile, ks, partials, cfg, ex, batch);
    if (vb == 4) return launch_tile<AK, BKC, 1, 4>(a, tile, ks, partials, cfg, ex, batch);
    return launch_tile<AK, BKC, 1, 1>(a, tile, ks, partials, cfg, ex, batch);
}

static cudaError_t launch_simt_any(const GemmArgs& a, int va, int vb, int tile, KSplit ks, float* partials, gemm_config_t* cfg,
                                   const SimtExtra& ex, int64_t batch) {
    cfg->kernel = GEMM_KERNEL_SIMT_FAST;
    cfg->split_k = ks.splits;
    cfg->vector_a = va; cfg->vector_b = vb;
    // A is contiguous along k when transposed; B is contiguous along k when not transposed
    if (!a.ta && (!a.tb || a.conv)) return launch_vec<false, true>(a, va, vb, tile, ks, partials, cfg, ex, batch);
    if (a.ta && (!a.tb || a.conv)) return launch_vec<true, true>(a, va, vb, tile, ks, partials, cfg, ex, batch);
    if (!a.ta && a.tb) return launch_vec<false, false>(a, va, vb, tile, ks, partials, cfg, ex, batch);
    return launch_vec<true, false>(a, va, vb, tile, ks, partials, cfg, ex, batch);
}

cudaError_t launch_simt_fast(const GemmArgs& a, int tile, KSplit ks, float* partials, gemm_config_t* cfg, TailSplit tail,
                             bool cluster_reduce) {
    int va, vb;
    simt_fast_eligible(a, &va, &vb);
    if (a.conv != nullptr)      // 128-bit loads need whole groups of four channels on 16-byte boundaries
        vb = ((reinterpret_cast<uintptr_t>(a.conv->X) & 15) == 0 && a.conv->c_in % 4 == 0) ? 4 : 1;
    const bool cluster = cluster_reduce && ks.splits > 1 && ks.splits <= CLUSTER_REDUCE_MAX_SPLITS && simt_fast_can_cluster_reduce(tile);
    if (cluster_reduce && !cluster) return cudaErrorInvalidConfiguration;
    const SimtExtra ex{tail, cluster ? 1 : 0, 0, 0, 0};
    return launch_simt_any(a, va, vb, tile, ks, cluster ? nullptr : partials, cfg, ex, 1);
}

cudaError_t launch_simt_fast_batched(const GemmArgs& a, int tile, int64_t strideA, int64_t strideB, int64_t strideC,
                                     int64_t batch, gemm_config_t* cfg) {
    int va, vb;
    simt_fast_eligible(a, &va, &vb);
    if (strideA % 4 != 0) va = 1;      // every problem's operands must keep the 16-byte alignment of the first
    if (strideB % 4 != 0) vb = 1;
    const SimtExtra ex{TailSplit{0x7FFFFFFF, 1, 0, nullptr}, 0, strideA, strideB, strideC};
    const KSplit whole{1, ((a.k > 0 ? a.k : 1) + BK - 1) / BK * BK};
    return launch_simt_any(a, va, vb, tile, whole, nullptr, cfg, ex, batch);
}

}  // namespace b200gemm
