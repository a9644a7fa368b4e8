// fp16 / bf16 GEMM with fp32 accumulation on the 5th-generation tensor cores (tcgen05, sm_100a).
//
// Mapping of the paper's algorithm (Fig. 1) onto the SM:
//   loops L1/L3 (jc, ic)   -> persistent CTAs walk a list of 128 x BN tiles of C (grouped so that resident CTAs
//                             share operand panels in L2)
//   loop  L2 (pc, kc)      -> 64-wide k blocks streamed through a multi-stage shared-memory ring
//   Pack-A / Pack-B        -> TMA copies global -> 128-byte-swizzled shared memory; the swizzled stage IS the
//                             packed panel, and TMA's zero fill past the matrix edge is the panel padding
//   loops L4/L5 + L6       -> tcgen05.mma 128 x BN x 16, issued by one thread; the C block lives in tensor
//                             memory (TMEM) for the whole k loop, as the paper's C block lives in registers
//   alpha / beta (Fig. 3)  -> epilogue warps read TMEM (tcgen05.ld), scale, and store column-major C
// Warp roles: warp 0 = TMA producer, warp 1 = MMA issuer + TMEM owner, warps 2..9 = epilogue (two per TMEM lane
// quarter, alternating 32-column chunks).  Two to four accumulators in TMEM let the epilogue of one tile overlap the
// main loops of the next ones.
// Every mbarrier wait is bounded: on expiry the role records a code in the status word and all roles drain.
#include <atomic>
#include <mutex>

#include "tc_common.cuh"

namespace b200gemm {

template <int BN> struct TcCfg {
    static constexpr int A_BYTES = TBM * TBK * 2;
    static constexpr int B_BYTES = BN * TBK * 2;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    // 227 KB of shared memory hold the operand ring plus the epilogue's staging tiles (one or two per warp)
    static constexpr int STAGES = (BN == 256) ? 4 : (BN == 128 ? 5 : 6);
    static constexpr int STORE_BUFS = (BN == 256) ? 1 : 2;
    static constexpr int NACC = (BN == 256) ? 2 : 4;               // accumulators in flight between MMA and epilogue
    static constexpr int TMEM_COLS = NACC * BN;                    // 512 columns per SM
    static constexpr int STORE_BYTES = EPI_WARPS * STORE_BUFS * 32 * 32 * 4;   // per epilogue warp: STORE_BUFS 32 x 32 fp32 tiles
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STORE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

// A_MN: op(A) is contiguous along m in memory (transA = N); B_MN: op(B) contiguous along n (transB = T).
// CONV: op(B) is the im2row-lowered activation matrix of a convolution layer, fetched by TMA in im2col mode
// straight from the NHWC tensor (tmB is then an im2col map); the lowered matrix never exists in memory.
// Split k summed by the cluster (see the kernel): this CTA's share of the BN-column tile whose partial sums lie, as dense
// [BN][128] fp32 tiles, at shared-memory offset `park_addr` of every CTA of the cluster.  Kept out of line so that its
// registers do not count against the main loop and the epilogue.
template <int BN>
__device__ __noinline__ void cluster_sum_tile(uint32_t park_addr, int S, int64_t row0, int64_t col0, int64_t m, int64_t n,
                                              float alpha, float beta, float* __restrict__ C, int64_t ldc, int out16) {
    const uint32_t rank = cluster_ctarank();
    constexpr int VECS = TBM * BN / 4;
    const int share = (VECS + S - 1) / S;
    const int v_end = min(VECS, (int)(rank + 1) * share);
    const bool cvec = !out16 && (reinterpret_cast<uintptr_t>(C) & 15) == 0 && ldc % 4 == 0;
    for (int v4 = (int)rank * share + (int)threadIdx.x; v4 < v_end; v4 += TC_THREADS) {
        const int e = v4 * 4, r = e % TBM, c = e / TBM;
        float4 q[8];
#pragma unroll
        for (int z = 0; z < 8; ++z)
            if (z < S) {
                const uint32_t ra = map_to_cta(park_addr + (uint32_t)e * 4u, (uint32_t)z);
                asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(q[z].x), "=f"(q[z].y), "=f"(q[z].z), "=f"(q[z].w) : "r"(ra));
            }
        float4 s4 = q[0];
#pragma unroll
        for (int z = 1; z < 8; ++z)
            if (z < S) { s4.x += q[z].x; s4.y += q[z].y; s4.z += q[z].z; s4.w += q[z].w; }
        const int64_t gi = row0 + r, gj = col0 + c;
        if (gi >= m || gj >= n) continue;
        const int64_t e0 = gi + gj * ldc;
        if (cvec && gi + 3 < m) {
            float4 o = make_float4(alpha * s4.x, alpha * s4.y, alpha * s4.z, alpha * s4.w);
            if (beta != 0.0f) {
                const float4 c0 = *reinterpret_cast<const float4*>(C + e0);
                o.x = fmaf(beta, c0.x, o.x); o.y = fmaf(beta, c0.y, o.y);
                o.z = fmaf(beta, c0.z, o.z); o.w = fmaf(beta, c0.w, o.w);
            }
            *reinterpret_cast<float4*>(C + e0) = o;
        } else {
            const float sv[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (gi + u < m) {
                    float o = alpha * sv[u];
                    if (beta != 0.0f) o = fmaf(beta, load_c(C, out16, e0 + u), o);
                    store_c(C, out16, e0 + u, o);
                }
        }
    }
}

// OUT: 0 = fp32 result; 1 = 16-bit result (fp32 accumulator, one rounding at the store); 2 = binary16 accumulator
// and binary16 result (the paper's all-f16 arithmetic, Section III-D); 3 = fp32 result stored transposed (the host
// exchanged the roles of the operands: C is ldc-strided along the tile's rows and contiguous along its columns)
template <int BN, bool A_MN, bool B_MN, bool CONV, int OUT, bool BATCHED>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmC, int store_via_tma, int64_t m, int64_t n, int64_t k, float alpha, float beta, float* __restrict__ C, int64_t ldc,
               int tiles_m, int tiles_n, int splits, int64_t kchunk, float* __restrict__ partials,
               uint32_t idesc, uint32_t* status, const ConvTma conv, int out16, int cluster_k, int batched,
               int64_t batch_c_bytes) {
    // BATCHED (then batched != 0): a strided batch of problems.  `splits` is then the number of problems and the slab index of a work
    // item the problem index: tmA and tmB are 3-D maps with the problem as third coordinate (bit 1 / bit 2 of `batched`:
    // A / B is one matrix shared by all problems), every item runs over the whole of k, and problem p's result starts
    // batch_c_bytes * p behind C.
    using Cfg = TcCfg<BN>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr bool OUT16 = OUT == 1 || OUT == 2, ACC16 = OUT == 2, CT = OUT == 3;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    // layout: [stages][C staging tiles of the epilogue warps][barriers]
    float* store_stage = reinterpret_cast<float*>(smem_al + STAGES * Cfg::STAGE_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * Cfg::STAGE_BYTES + Cfg::STORE_BYTES);
    // barrier slots: [0,S) full, [S,2S) empty, then NACC tmem_full, NACC tmem_empty, then 2 words
    const uint32_t bar0 = smem_base + STAGES * Cfg::STAGE_BYTES + Cfg::STORE_BYTES;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    constexpr int NACC = Cfg::NACC;
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + NACC + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 2 * STAGES + 2 * NACC);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // let the next kernel of the stream start its own set-up as soon as SMs free up (it waits before touching memory)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 32) {      // descriptors into the TMA unit's cache while the barriers are set up
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        if (store_via_tma) prefetch_tensormap(&tmC);
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < NACC; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), EPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // TMEM allocation is a warp-wide operation; the base address lands in shared memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Programmatic dependent launch: everything above (barrier and TMEM set-up) may overlap the tail of the
    // previous kernel in the stream; nothing below touches global memory before that kernel has completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const int64_t items = (int64_t)tiles_m * tiles_n * splits;
    // Work items of this CTA.  Ordinarily: blockIdx.x, blockIdx.x + gridDim.x, ...  With cluster_k (split k finished
    // inside the kernel) every CTA has exactly one item: the cluster is the tile, the rank in the cluster the k range.
    int64_t item_first = blockIdx.x, item_step = gridDim.x;
    if (cluster_k) {
        item_first = (int64_t)(blockIdx.x % cluster_k) * ((int64_t)tiles_m * tiles_n) + blockIdx.x / cluster_k;
        item_step = items;
    }
    constexpr int GROUP = 16;
    auto decode = [&](int64_t item, int& tm, int& tn, int& sp) {
        const int64_t tiles = (int64_t)tiles_m * tiles_n;
        sp = (int)(item / tiles);
        const int tile = (int)(item % tiles);
        const int per_group = GROUP * tiles_n;
        const int g = tile / per_group;
        const int gsz = min(GROUP, tiles_m - g * GROUP);
        tm = g * GROUP + (tile % per_group) % gsz;
        tn = (tile % per_group) / gsz;
    };
    auto kblocks_of = [&](int sp, int64_t& kbeg) {
        if (BATCHED) { kbeg = 0; return (int)((k + TBK - 1) / TBK); }
        kbeg = (int64_t)sp * kchunk;
        const int64_t kend = min(k, kbeg + kchunk);
        return (int)((kend - kbeg + TBK - 1) / TBK);
    };

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t cnt = 0;
            bool ok = true;
            for (int64_t item = item_first; item < items && ok; item += item_step) {
                int tm, tn, sp;
                decode(item, tm, tn, sp);
                int64_t kbeg;
                const int kb_n = kblocks_of(sp, kbeg);
                const int32_t m0 = tm * TBM, n0 = tn * BN;
                int32_t cw = 0, ch = 0, cn = 0;
                if (CONV) conv_tile_origin(conv, (int64_t)tn * BN, cw, ch, cn);
                for (int kb = 0; kb < kb_n; ++kb, ++cnt) {
                    const int s = cnt % STAGES;
                    const uint32_t ph = (cnt / STAGES) & 1;
                    if (!mbar_wait(empty_bar(s), ph ^ 1, abort_flag, status,
                                   STATUS_MARK | (ROLE_TMA << 16) | (BAR_EMPTY << 8) | s)) { ok = false; break; }
                    const uint32_t sa = smem_base + s * Cfg::STAGE_BYTES;
                    const uint32_t sb = sa + Cfg::A_BYTES;
                    const int32_t k0 = (int32_t)(kbeg + (int64_t)kb * TBK);
                    mbar_expect_tx(full_bar(s), Cfg::STAGE_BYTES);
                    if constexpr (BATCHED) {
                        const int32_t pa = (batched & 2) ? 0 : sp, pb = (batched & 4) ? 0 : sp;
                        if (A_MN) {
#pragma unroll
                            for (int c = 0; c < TBM / 64; ++c)
                                tma_load_3d(&tmA, sa + c * (64 * TBK * 2), full_bar(s), m0 + c * 64, k0, pa);
                        } else {
                            tma_load_3d(&tmA, sa, full_bar(s), k0, m0, pa);
                        }
                        if (B_MN) {
#pragma unroll
                            for (int c = 0; c < BN / 64; ++c)
                                tma_load_3d(&tmB, sb + c * (64 * TBK * 2), full_bar(s), n0 + c * 64, k0, pb);
                        } else {
                            tma_load_3d(&tmB, sb, full_bar(s), k0, n0, pb);
                        }
                        continue;
                    }
                    if (A_MN) {
#pragma unroll
                        for (int c = 0; c < TBM / 64; ++c) tma_load_2d(&tmA, sa + c * (64 * TBK * 2), full_bar(s), m0 + c * 64, k0);
                    } else {
                        tma_load_2d(&tmA, sa, full_bar(s), k0, m0);
                    }
                    if (CONV) {
                        const int kg = k0 / TBK;                     // k block -> filter tap and channel chunk
                        const int tap = kg / conv.chunks, c0 = (kg - tap * conv.chunks) * TBK;
                        const int fr = tap / conv.kw, fs = tap - fr * conv.kw;
                        tma_load_im2col(&tmB, sb, full_bar(s), c0, cw, ch, cn, (uint16_t)fs, (uint16_t)fr);
                    } else if (B_MN) {
#pragma unroll
                        for (int c = 0; c < BN / 64; ++c) tma_load_2d(&tmB, sb + c * (64 * TBK * 2), full_bar(s), n0 + c * 64, k0);
                    } else {
                        tma_load_2d(&tmB, sb, full_bar(s), k0, n0);
                    }
                }
            }
            // drain: do not leave the CTA while copies that were armed may still be landing
            const uint32_t armed = cnt < (uint32_t)STAGES ? cnt : (uint32_t)STAGES;
            for (uint32_t i = 0; i < armed; ++i) {
                const uint32_t c = cnt - 1 - i;
                const int s = c % STAGES;
                const uint32_t ph = (c / STAGES) & 1;
                for (uint32_t it = 0; it < (1u << 20); ++it)
                    if (mbar_try_wait(full_bar(s), ph)) break;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t cnt = 0, it = 0;
            bool ok = true;
            for (int64_t item = item_first; item < items && ok; item += item_step, ++it) {
                int tm, tn, sp;
                decode(item, tm, tn, sp);
                int64_t kbeg;
                const int kb_n = kblocks_of(sp, kbeg);
                const uint32_t acc = it % NACC, aph = (it / NACC) & 1;
                if (!mbar_wait(tempty_bar(acc), aph ^ 1, abort_flag, status,
                               STATUS_MARK | (ROLE_MMA << 16) | (BAR_TMEM_EMPTY << 8) | acc)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < kb_n; ++kb, ++cnt) {
                    const int s = cnt % STAGES;
                    const uint32_t ph = (cnt / STAGES) & 1;
                    if (!mbar_wait(full_bar(s), ph, abort_flag, status,
                                   STATUS_MARK | (ROLE_MMA << 16) | (BAR_FULL << 8) | s)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_base + s * Cfg::STAGE_BYTES;
                    const uint32_t sb = sa + Cfg::A_BYTES;
#pragma unroll
                    for (int kk = 0; kk < TBK / UMMA_K; ++kk) {
                        // K-major: 16 k = 32 bytes inside the 128-byte row.  MN-major: 16 k rows of 128 bytes;
                        // 64-element chunks of m/n are TBK*128 bytes apart, 8-row k groups 1024 bytes apart.
                        const uint64_t ad = A_MN ? smem_desc(sa + kk * (UMMA_K * 128), TBK * 128, 1024)
                                                 : smem_desc(sa + kk * (UMMA_K * 2), 0, 1024);
                        const uint64_t bd = B_MN ? smem_desc(sb + kk * (UMMA_K * 128), TBK * 128, 1024)
                                                 : smem_desc(sb + kk * (UMMA_K * 2), 0, 1024);
                        umma_f16(d_tmem, ad, bd, idesc, (kb | kk) != 0);
                    }
                    umma_commit(empty_bar(s));          // frees the stage when these MMAs have read it
                }
                if (!ok) break;
                umma_commit(tfull_bar(acc));            // accumulator complete
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..9), TMEM lanes 32q .. 32q+31
        // Lane = row of C.  Each 32-column chunk is read from TMEM, scaled, and then either written straight to
        // global memory (a warp stores 32 consecutive floats of one column per instruction) or, when C can be
        // addressed by TMA, transposed through a 32 x 32 staging tile in shared memory and written by an
        // asynchronous bulk tensor store, which also clips the tile at the matrix edge.
        const int q = warp & 3;                       // a warp may touch TMEM lanes 32*(warp % 4) .. +31 only
        const int half = (warp - 2) >> 2;             // which of the two warps of this lane quarter
        float* stage = store_stage + (warp - 2) * (Cfg::STORE_BUFS * 32 * 32);
        uint32_t it = 0, sbuf = 0;
        bool ok = true;
        for (int64_t item = item_first; item < items && ok; item += item_step, ++it) {
            int tm, tn, sp;
            decode(item, tm, tn, sp);
            const uint32_t acc = it % NACC, aph = (it / NACC) & 1;
            if (!mbar_wait(tfull_bar(acc), aph, abort_flag, status,
                           STATUS_MARK | (ROLE_EPI << 16) | (BAR_TMEM_FULL << 8) | acc)) { ok = false; break; }
            tc_fence_after();
            const int64_t row0 = (int64_t)tm * TBM + q * 32;
            const bool raw = splits > 1 && !BATCHED;
            float* out = raw ? partials + (int64_t)sp * m * n : C;
            if (BATCHED) out = reinterpret_cast<float*>(reinterpret_cast<char*>(C) + (int64_t)sp * batch_c_bytes);
            // store_via_tma: 0 = direct stores, 1 = tmC maps C (2-D), 2 = tmC maps the split-k partials (3-D: m, n, split)
            const bool via_tma = raw ? (store_via_tma == 2) : (store_via_tma == 1);
            auto release = [&]() {      // the accumulator may be overwritten once this warp has read its last chunk
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(tempty_bar(acc));
            };
            const uint32_t tacc = tmem_base + acc * BN + ((uint32_t)(q * 32) << 16);
            if (cluster_k) {
                // park the raw accumulator in shared memory as a dense [BN][128] fp32 tile (the operand stages are free:
                // every MMA that read them has completed); the cluster sums it below
                float* park = reinterpret_cast<float*>(smem_al);
#pragma unroll 1
                for (int c = half; c < BN / 32; c += 2) {
                    uint32_t v[32];
                    tmem_ld32(tacc + c * 32, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) park[(c * 32 + j) * TBM + q * 32 + lane] = __uint_as_float(v[j]);
                }
                release();
                continue;
            }
            bool done = false;
            if constexpr (CT) {
                epilogue_tile_ct<BN, Cfg::STORE_BUFS>(tacc, row0, (int64_t)tn * BN, half, lane, m, n, alpha, beta, C, ldc,
                                                      store_via_tma == 3, &tmC, stage, sbuf, release);
                done = true;
            }
            if constexpr (OUT16) {
                if (!raw) {      // 16-bit result: one rounding at the store (split-k partial sums stay fp32)
                    epilogue_tile16<BN, Cfg::STORE_BUFS, ACC16>(tacc, row0, (int64_t)tn * BN, half, lane, m, n, alpha, beta, out, ldc,
                                                store_via_tma == 1, &tmC, stage, sbuf, out16, release);
                    done = true;
                }
            }
            if (!done)
                epilogue_tile<BN, Cfg::STORE_BUFS>(tacc, row0, (int64_t)tn * BN, half, lane, m, n, alpha, beta, out, raw ? m : ldc,
                                          raw, via_tma, &tmC, sp, stage, sbuf, release);
        }
        if (lane == 0) bulk_wait_all();       // staging tiles must outlive the stores that read them
    }

    if (cluster_k) {
        // ------------------------------------------------ split k summed by the cluster (every thread of every CTA)
        // Each CTA of the cluster holds the partial sums of its k range in shared memory.  After a cluster barrier this
        // CTA sums a contiguous share of the tile over all CTAs, in increasing k range whoever does the summing,
        // through distributed shared memory, applies alpha / beta and writes C.  The barrier is the hardware's (a
        // cluster is co-scheduled); a role that gave up a bounded wait arrives here as well, so nobody waits in vain.
        __syncthreads();
        __syncwarp();
        cluster_sync_all();
        if (*abort_flag == 0) {
            int tm, tn, sp;
            decode(item_first, tm, tn, sp);
            cluster_sum_tile<BN>(smem_base, cluster_k, (int64_t)tm * TBM, (int64_t)tn * BN, m, n, alpha, beta, C, ldc, out16);
        }
        __syncwarp();
        cluster_sync_all();      // nobody leaves while its shared memory may still be read
    }

    // ------------------------------------------------ teardown: every thread arrives here on every path
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
    }
}

// Self-test of the give-up path: one thread waits, with a short limit, on a barrier that nothing ever arrives at.
// The wait expires, the code lands in the status word and the kernel returns normally.
__global__ void __launch_bounds__(32) wait_expiry_probe_kernel(uint32_t* status, uint32_t limit) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        mbar_wait(smem_u32(&bar), 0, &abort_flag, status, STATUS_MARK | (ROLE_SELFTEST << 16) | (BAR_FULL << 8), limit);
    }
    __syncthreads();
}

cudaError_t launch_wait_expiry_probe(uint32_t* status, cudaStream_t stream) {
    wait_expiry_probe_kernel<<<1, 32, 0, stream>>>(status, SPIN_FAST + 2048);     // a few hundred microseconds
    return cudaGetLastError();
}

// ---------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;           // several host threads may make their first 16-bit call at the same time
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// Tensor maps are pure functions of what they describe (address, type, extents, stride, box), and encoding one costs
// the host about a microsecond.  Each host thread keeps the last few it built: a caller that multiplies the same
// buffers again (the usual case: a layer's weights, a pre-allocated activation buffer) gets its maps from here.
struct MapKey {
    uint64_t v[7];
    bool operator==(const MapKey& o) const {
        for (int i = 0; i < 7; ++i)
            if (v[i] != o.v[i]) return false;
        return true;
    }
};
struct MapCache {
    static constexpr int N = 32;
    MapKey key[N];
    CUtensorMap map[N];
    bool used[N] = {};
    int next = 0;
};
template <typename Encode>
static bool cached_map(CUtensorMap* tm, const MapKey& k, Encode&& encode) {
    static thread_local MapCache cache;
    for (int i = 0; i < MapCache::N; ++i)
        if (cache.used[i] && cache.key[i] == k) { *tm = cache.map[i]; return true; }
    if (!encode(tm)) return false;
    const int slot = cache.next;
    cache.next = (cache.next + 1) % MapCache::N;
    cache.key[slot] = k;
    cache.map[slot] = *tm;
    cache.used[slot] = true;
    return true;
}

// 2-D map over a stored column-major matrix: dim0 = contiguous dimension (rows), dim1 = columns (stride ld)
bool make_map(CUtensorMap* tm, int dtype, const void* base, int64_t rows, int64_t cols, int64_t ld,
                     uint32_t box_rows, uint32_t box_cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const MapKey k{{1, (uint64_t)dtype, (uint64_t)(uintptr_t)base, (uint64_t)rows, (uint64_t)cols, (uint64_t)ld,
                    ((uint64_t)box_rows << 32) | box_cols}};
    return cached_map(tm, k, [&](CUtensorMap* out) {
        cuuint64_t dims[2] = {(cuuint64_t)rows, (cuuint64_t)cols};
        cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
        cuuint32_t box[2] = {box_rows, box_cols};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = fn(out, dtype == GEMM_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                        const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        return r == CUDA_SUCCESS;
    });
}

bool make_map_batched(CUtensorMap* tm, int dtype, const void* base, int64_t rows, int64_t cols, int64_t ld, int64_t stride,
                      int64_t batch, uint32_t box_rows, uint32_t box_cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    if (batch > 1 && (stride <= 0 || stride % 8 != 0)) return false;
    if (batch <= 1) stride = ld * (cols > 0 ? cols : 1);      // a single problem: any legal value
    if (rows > 0xFFFFFFFFLL || cols > 0xFFFFFFFFLL || box_rows > 0xFFFF || box_cols > 0xFFFF) return false;
    const MapKey k{{5, (uint64_t)dtype | ((uint64_t)box_rows << 16) | ((uint64_t)box_cols << 32), (uint64_t)(uintptr_t)base,
                    ((uint64_t)rows << 32) | (uint64_t)cols, (uint64_t)ld, (uint64_t)stride, (uint64_t)batch}};
    return cached_map(tm, k, [&](CUtensorMap* out) {
        cuuint64_t dims[3] = {(cuuint64_t)rows, (cuuint64_t)cols, (cuuint64_t)batch};
        cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)stride * 2};
        cuuint32_t box[3] = {box_rows, box_cols, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = fn(out, dtype == GEMM_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                        const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        return r == CUDA_SUCCESS;
    });
}

// map over the split-k partial sums [split][n][m] (fp32, dense): 32 x 32 x 1 boxes
bool make_partials_map(CUtensorMap* tm, const float* base, int64_t m, int64_t n, int splits) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const MapKey k{{2, 0, (uint64_t)(uintptr_t)base, (uint64_t)m, (uint64_t)n, (uint64_t)splits, 0}};
    return cached_map(tm, k, [&](CUtensorMap* out) {
        cuuint64_t dims[3] = {(cuuint64_t)m, (cuuint64_t)n, (cuuint64_t)splits};
        cuuint64_t strides[2] = {(cuuint64_t)m * 4, (cuuint64_t)m * (cuuint64_t)n * 4};
        cuuint32_t box[3] = {32, 32, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        return r == CUDA_SUCCESS;
    });
}

// map over the result (fp32 or a 16-bit type) for the epilogue's tile stores: 32 x 32 boxes, no swizzle
bool make_c_map(CUtensorMap* tm, const float* base, int64_t m, int64_t n, int64_t ldc, int out16) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const MapKey k{{3, (uint64_t)out16, (uint64_t)(uintptr_t)base, (uint64_t)m, (uint64_t)n, (uint64_t)ldc, 0}};
    return cached_map(tm, k, [&](CUtensorMap* out) {
        cuuint64_t dims[2] = {(cuuint64_t)m, (cuuint64_t)n};
        cuuint64_t strides[1] = {(cuuint64_t)ldc * (out16 ? 2 : 4)};
        const CUtensorMapDataType dt = out16 == GEMM_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                       : out16 == GEMM_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
        cuuint32_t box[2] = {32, 32};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = fn(out, dt, 2, const_cast<float*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        return r == CUDA_SUCCESS;
    });
}

bool make_ct_map(CUtensorMap* tm, const float* base, int64_t c_rows, int64_t c_cols, int64_t ldc) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const MapKey k{{4, 0, (uint64_t)(uintptr_t)base, (uint64_t)c_rows, (uint64_t)c_cols, (uint64_t)ldc, 0}};
    return cached_map(tm, k, [&](CUtensorMap* out) {
        cuuint64_t dims[2] = {(cuuint64_t)c_rows, (cuuint64_t)c_cols};
        cuuint64_t strides[1] = {(cuuint64_t)ldc * 4};
        cuuint32_t box[2] = {32, 32};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        return r == CUDA_SUCCESS;
    });
}

typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);

static EncodeIm2colFn encode_im2col_fn() {
    static EncodeIm2colFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeIm2colFn>(p);
    });
    return fn;
}

bool conv_tma_eligible(int dtype, const ConvIndex& cv, int64_t batch) {
    if (dtype != GEMM_F16 && dtype != GEMM_BF16) return false;
    if (cv.c_in % 64 != 0 || (reinterpret_cast<uintptr_t>(cv.X) & 15) != 0) return false;
    if (cv.kh != cv.kw || cv.sh != cv.sw || cv.ph != cv.pw) return false;      // one corner / stride value serves both directions
    if (cv.sh < 1 || cv.sh > 8 || cv.ph > 127 || cv.kh > 128 || cv.ph - (cv.kh - 1) < -128) return false;   // field ranges of the map
    if (cv.kh > 255) return false;                                             // filter offsets travel as 16-bit values
    if (cv.h > 0x7FFFFFFF || cv.w > 0x7FFFFFFF || batch > 0x7FFFFFFF) return false;
    if (cv.w * cv.c_in * 2 >= (1LL << 40) || cv.h * cv.w * cv.c_in * 2 >= (1LL << 40)) return false;
    return encode_im2col_fn() != nullptr;
}

bool make_im2col_map(CUtensorMap* tm, int dtype, const ConvIndex& cv, int64_t batch, uint32_t pixels) {
    EncodeIm2colFn fn = encode_im2col_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {(cuuint64_t)cv.c_in, (cuuint64_t)cv.w, (cuuint64_t)cv.h, (cuuint64_t)batch};
    cuuint64_t strides[3] = {(cuuint64_t)cv.c_in * 2, (cuuint64_t)cv.w * cv.c_in * 2, (cuuint64_t)cv.h * cv.w * cv.c_in * 2};
    // receptive-field corners may start at -pad and must stop where the last filter tap still touches image + pad
    int lower[2] = {-cv.pw, -cv.ph};
    int upper[2] = {cv.pw - (cv.kw - 1), cv.ph - (cv.kh - 1)};
    cuuint32_t estr[4] = {1, (cuuint32_t)cv.sw, (cuuint32_t)cv.sh, 1};
    CUresult r = fn(tm, dtype == GEMM_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
                    const_cast<void*>(cv.X), dims, strides, lower, upper, 64, pixels, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool tensor_eligible(const GemmArgs& a) {
    if (a.dtype != GEMM_F16 && a.dtype != GEMM_BF16) return false;
    auto ok = [](const void* p, int64_t ld) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0 && ld % 8 == 0; };
    if (!ok(a.A, a.lda) || !ok(a.B, a.ldb)) return false;
    if (a.m > 0x7FFFFFFFLL || a.n > 0x7FFFFFFFLL || a.k > 0x7FFFFFFFLL) return false;
    if (a.lda * 2 >= (1LL << 40) || a.ldb * 2 >= (1LL << 40)) return false;
    return encode_fn() != nullptr;
}

uint32_t instr_desc(int dtype, bool a_mn, bool b_mn, int mma_m, int mma_n, bool acc16) {
    const uint32_t fmt = dtype == GEMM_F16 ? 0u : 1u;    // input format: 0 = f16, 1 = bf16
    uint32_t d = 0;
    d |= (acc16 ? 0u : 1u) << 4;     // accumulator format: 1 = f32, 0 = f16
    d |= fmt << 7;                   // A format
    d |= fmt << 10;                  // B format
    d |= (a_mn ? 1u : 0u) << 15;     // A is MN-major
    d |= (b_mn ? 1u : 0u) << 16;     // B is MN-major
    d |= (uint32_t)(mma_n >> 3) << 17;  // N / 8
    d |= (uint32_t)(mma_m >> 4) << 24; // M / 16
    return d;
}

template <int BN, bool A_MN, bool B_MN, bool CONV, int OUT, bool BATCHED = false>
static cudaError_t launch_tc(const GemmArgs& a, KSplit ks, float* partials, gemm_config_t* cfg,
                             const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC, int store_via_tma,
                             bool cluster = false, int batched = 0, int64_t batch_c_bytes = 0) {
    using Cfg = TcCfg<BN>;
    // the opt-in to more than 48 KB of dynamic shared memory is per device
    static std::atomic<bool> attr_set[64];      // zero-initialised; set once per device
    auto kern = tc_gemm_kernel<BN, A_MN, B_MN, CONV, OUT, BATCHED>;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev].load()) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev].store(true);
    }
    const int64_t tiles_m = (a.m + TBM - 1) / TBM, tiles_n = (a.n + BN - 1) / BN;
    if (tiles_m > 0x7FFFFFFF || tiles_n > 0x7FFFFFFF || tiles_m * tiles_n > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const int64_t items = tiles_m * tiles_n * ks.splits;
    if (cluster && (ks.splits < 2 || ks.splits > 8 || items > 0x7FFFFFFFLL)) return cudaErrorInvalidConfiguration;
    // cluster: one CTA per item, the k ranges of a tile forming a cluster; otherwise a persistent grid
    const int grid = cluster ? (int)items : (int)(items < sm_count() ? items : sm_count());
    cfg->tile_m = TBM; cfg->tile_n = BN; cfg->tile_k = TBK; cfg->stages = Cfg::STAGES; cfg->grid = grid;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)grid);
    lc.blockDim = dim3(TC_THREADS);
    lc.dynamicSmemBytes = Cfg::SMEM_BYTES;
    lc.stream = a.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // pairs with griddepcontrol.wait in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (cluster) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)ks.splits;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        lc.numAttrs = 2;
    }
    cudaError_t le = cudaLaunchKernelEx(&lc, kern, tmA, tmB, tmC, store_via_tma, a.m, a.n, a.k, a.alpha, a.beta, a.C, a.ldc,
                                        (int)tiles_m, (int)tiles_n, ks.splits, ks.chunk,
                                        (ks.splits > 1 && !cluster) ? partials : (float*)nullptr,
                                        instr_desc(a.dtype, A_MN, B_MN, TBM, BN, OUT == 2), a.status, conv_tma_params(a.conv), a.out16,
                                        cluster ? ks.splits : 0, batched, batch_c_bytes);
    return le != cudaSuccess ? le : cudaGetLastError();
}

// A strided batch of 16-bit problems in one launch: 3-D maps of A and B (a shared operand, stride 0, keeps its 2-D
// extent with one problem in the third dimension), KSplit.splits carries the number of problems.
template <bool A_MN, bool B_MN>
static cudaError_t launch_tc_batched(const GemmArgs& a, int tile_n, int64_t strideA, int64_t strideB, int64_t strideC,
                                     int64_t batch, gemm_config_t* cfg) {
    if (batch < 1 || batch > 0x7FFFFFFFLL || a.conv || a.acc16 || a.ct) return cudaErrorInvalidConfiguration;
    CUtensorMap tmA, tmB;
    const int64_t na = strideA == 0 ? 1 : batch, nb = strideB == 0 ? 1 : batch;
    bool ok = A_MN ? make_map_batched(&tmA, a.dtype, a.A, a.m, a.k, a.lda, strideA, na, 64, TBK)
                   : make_map_batched(&tmA, a.dtype, a.A, a.k, a.m, a.lda, strideA, na, TBK, TBM);
    ok = ok && (B_MN ? make_map_batched(&tmB, a.dtype, a.B, a.n, a.k, a.ldb, strideB, nb, 64, TBK)
                     : make_map_batched(&tmB, a.dtype, a.B, a.k, a.n, a.ldb, strideB, nb, TBK, (uint32_t)tile_n));
    if (!ok) return cudaErrorInvalidValue;
    const int flags = 1 | (strideA == 0 ? 2 : 0) | (strideB == 0 ? 4 : 0);
    const int64_t c_bytes = strideC * (a.out16 ? 2 : 4);
    const KSplit ks{(int)batch, a.k};
    switch (tile_n) {
        case 256: return a.out16 ? launch_tc<256, A_MN, B_MN, false, 1, true>(a, ks, nullptr, cfg, tmA, tmB, tmA, 0, false, flags, c_bytes)
                                  : launch_tc<256, A_MN, B_MN, false, 0, true>(a, ks, nullptr, cfg, tmA, tmB, tmA, 0, false, flags, c_bytes);
        case 128: return a.out16 ? launch_tc<128, A_MN, B_MN, false, 1, true>(a, ks, nullptr, cfg, tmA, tmB, tmA, 0, false, flags, c_bytes)
                                  : launch_tc<128, A_MN, B_MN, false, 0, true>(a, ks, nullptr, cfg, tmA, tmB, tmA, 0, false, flags, c_bytes);
        default:  return a.out16 ? launch_tc<64, A_MN, B_MN, false, 1, true>(a, ks, nullptr, cfg, tmA, tmB, tmA, 0, false, flags, c_bytes)
                                  : launch_tc<64, A_MN, B_MN, false, 0, true>(a, ks, nullptr, cfg, tmA, tmB, tmA, 0, false, flags, c_bytes);
    }
}

cudaError_t launch_tensor_batched(const GemmArgs& a, int tile_n, int64_t strideA, int64_t strideB, int64_t strideC,
                                  int64_t batch, gemm_config_t* cfg) {
    cfg->kernel = GEMM_KERNEL_TENSOR;
    cfg->split_k = 1;
    cfg->vector_a = cfg->vector_b = 1;
    const bool a_mn = !a.ta, b_mn = a.tb;
    if (a_mn && b_mn) return launch_tc_batched<true, true>(a, tile_n, strideA, strideB, strideC, batch, cfg);
    if (a_mn && !b_mn) return launch_tc_batched<true, false>(a, tile_n, strideA, strideB, strideC, batch, cfg);
    if (!a_mn && b_mn) return launch_tc_batched<false, true>(a, tile_n, strideA, strideB, strideC, batch, cfg);
    return launch_tc_batched<false, false>(a, tile_n, strideA, strideB, strideC, batch, cfg);
}

template <bool A_MN, bool B_MN, bool CONV>
static cudaError_t launch_tc_bn(const GemmArgs& a, int tile_n, KSplit ks, float* partials, gemm_config_t* cfg, bool cluster) {
    CUtensorMap tmA, tmB;
    // stored A: (m x k) if transA = N [contiguous m], (k x m) otherwise [contiguous k]
    bool ok = A_MN ? make_map(&tmA, a.dtype, a.A, a.m, a.k, a.lda, 64, TBK)
                   : make_map(&tmA, a.dtype, a.A, a.k, a.m, a.lda, TBK, TBM);
    // stored B: (k x n) if transB = N [contiguous k], (n x k) otherwise [contiguous n]
    if (CONV) {      // n = batch * Ho * Wo pixels
        ok = ok && make_im2col_map(&tmB, a.dtype, *a.conv, a.n / ((int64_t)a.conv->ho * a.conv->wo), (uint32_t)tile_n);
    } else {
        ok = ok && (B_MN ? make_map(&tmB, a.dtype, a.B, a.n, a.k, a.ldb, 64, TBK)
                         : make_map(&tmB, a.dtype, a.B, a.k, a.n, a.ldb, TBK, (uint32_t)tile_n));
    }
    if (!ok) return cudaErrorInvalidValue;
    // the result goes out through TMA tile stores when C is 16-byte addressable and this is not a split-k pass
    CUtensorMap tmC = tmA;
    int store_via_tma = 0;
    if (!a.ct && ks.splits == 1 && c_tma_addressable(a.C, a.m, a.ldc, a.out16))
        store_via_tma = make_c_map(&tmC, a.C, a.m, a.n, a.ldc, a.out16) ? 1 : 0;
    if (ks.splits > 1 && !cluster && (reinterpret_cast<uintptr_t>(partials) & 15) == 0 && a.m % 4 == 0 &&
        a.m * a.n * 4 < (1LL << 40))
        store_via_tma = make_partials_map(&tmC, partials, a.m, a.n, ks.splits) ? 2 : 0;
    if constexpr (!CONV) {
        if (a.ct) {      // operands exchanged by the host: n (the caller's m) is at most 64, C goes out transposed
            if (tile_n != 64 || ks.splits != 1 || a.out16) return cudaErrorInvalidConfiguration;
            // here a.n is the row count of the caller's C and a.m its column count; tile stores when C is 16-byte addressable
            int ct_store = 0;
            if (c_tma_addressable(a.C, a.n, a.ldc, 0) && make_ct_map(&tmC, a.C, a.n, a.m, a.ldc)) ct_store = 3;
            return launch_tc<64, A_MN, B_MN, false, 3>(a, ks, partials, cfg, tmA, tmB, tmC, ct_store);
        }
        if (a.acc16) {      // binary16 accumulator (never split along k: partial sums would need a wider type)
            switch (tile_n) {
                case 256: return launch_tc<256, A_MN, B_MN, false, 2>(a, ks, partials, cfg, tmA, tmB, tmC, store_via_tma);
                case 128: return launch_tc<128, A_MN, B_MN, false, 2>(a, ks, partials, cfg, tmA, tmB, tmC, store_via_tma);
                default:  return launch_tc<64, A_MN, B_MN, false, 2>(a, ks, partials, cfg, tmA, tmB, tmC, store_via_tma);
            }
        }
    }
    switch (tile_n) {
        case 256: return a.out16 ? launch_tc<256, A_MN, B_MN, CONV, 1>(a, ks, partials, cfg, tmA, tmB, tmC, store_via_tma, cluster)
                                  : launch_tc<256, A_MN, B_MN, CONV, 0>(a, ks, partials, cfg, tmA, tmB, tmC, store_via_tma, cluster);
        case 128: return a.out16 ? launch_tc<128, A_MN, B_MN, CONV, 1>(a, ks, partials, cfg, tmA, tmB, tmC, store_via_tma, cluster)
                                  : launch_tc<128, A_MN, B_MN, CONV, 0>(a, ks, partials, cfg, tmA, tmB, tmC, store_via_tma, cluster);
        default:  return a.out16 ? launch_tc<64, A_MN, B_MN, CONV, 1>(a, ks, partials, cfg, tmA, tmB, tmC, store_via_tma, cluster)
                                  : launch_tc<64, A_MN, B_MN, CONV, 0>(a, ks, partials, cfg, tmA, tmB, tmC, store_via_tma, cluster);
    }
}

cudaError_t launch_tensor(const GemmArgs& a, int tile_n, KSplit ks, float* partials, gemm_config_t* cfg, bool cluster) {
    cfg->kernel = GEMM_KERNEL_TENSOR;
    cfg->split_k = ks.splits;
    cfg->vector_a = cfg->vector_b = 1;
    const bool a_mn = !a.ta, b_mn = a.tb;
    if (a.conv != nullptr)
        return a_mn ? launch_tc_bn<true, false, true>(a, tile_n, ks, partials, cfg, cluster)
                    : launch_tc_bn<false, false, true>(a, tile_n, ks, partials, cfg, cluster);
    if (a_mn && b_mn) return launch_tc_bn<true, true, false>(a, tile_n, ks, partials, cfg, cluster);
    if (a_mn && !b_mn) return launch_tc_bn<true, false, false>(a, tile_n, ks, partials, cfg, cluster);
    if (!a_mn && b_mn) return launch_tc_bn<false, true, false>(a, tile_n, ks, partials, cfg, cluster);
    return launch_tc_bn<false, false, false>(a, tile_n, ks, partials, cfg, cluster);
}

}  // namespace b200gemm
