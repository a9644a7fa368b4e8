// fp16 / bf16 GEMM on CTA pairs: two SMs work on one 256 x 256 tile of C (tcgen05 cta_group::2).
//
// Same mapping of the paper's algorithm (Fig. 1) as the single-CTA tensor kernel, with the C block of the
// micro-kernel doubled in m: the pair's tile is 256 rows x 256 columns, CTA r of the pair owns rows 128 r .. 128 r + 127
// (its 128 TMEM lanes x 256 columns).  Each CTA stages only its own 128 rows of op(A) and its own 128 of the tile's
// 256 columns of op(B); one tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 16), issued by a single thread of the
// leader CTA (rank 0), reads A from each CTA's own shared memory and the two halves of B from both.  Per k block a
// CTA therefore fills 32 KB of shared memory for 128 x 256 of output instead of 48 KB: the stage fill rate, which
// limits the single-CTA kernel, is cut by a third, and six stages fit where four did.
//
// Synchronisation (all waits bounded, as everywhere in this library):
//   full[s]    leader only; both CTAs' TMA copies complete their bytes on it (copies carry the cta_group::2 form,
//              whose mbarrier may live in the peer CTA); the leader's producer posts the expected byte count
//   empty[s]   one per CTA; the leader's tcgen05.commit arrives on both (commit with a CTA mask) once the MMAs
//              that read the stage have completed
//   tfull[a]   one per CTA; same commit form, when the accumulator of a tile is complete
//   tempty[a]  leader only; the epilogue warps of both CTAs arrive (the peer's through the cluster address)
// No TMA load here is multicast: every CTA fetches what it stages itself.
#include <atomic>

#include "tc_common.cuh"

namespace b200gemm {

constexpr int PAIR_BN = 256;                 // columns of the pair's tile = N of the MMA
constexpr int PAIR_HALF_N = PAIR_BN / 2;     // columns of op(B) staged by one CTA
constexpr int PAIR_STAGES = 6;
constexpr int PAIR_NACC = 2;                 // 2 x 256 TMEM columns
constexpr int PAIR_A_BYTES = TBM * TBK * 2;
constexpr int PAIR_B_BYTES = PAIR_HALF_N * TBK * 2;
constexpr int PAIR_STAGE_BYTES = PAIR_A_BYTES + PAIR_B_BYTES;                  // per CTA
constexpr int PAIR_STORE_BYTES = EPI_WARPS * 32 * 32 * 4;
constexpr int PAIR_SMEM_BYTES = PAIR_STAGES * PAIR_STAGE_BYTES + PAIR_STORE_BYTES + 1024 + 256;

// CONV: op(B) is the lowered activation matrix of a convolution layer, fetched in im2col mode (see tc_gemm.cu)
template <bool A_MN, bool B_MN, bool CONV, bool OUT16>
__global__ void __launch_bounds__(TC_THREADS, 1)
tc_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmC, int store_via_tma, int64_t m, int64_t n, int64_t k,
                    float alpha, float beta, float* __restrict__ C, int64_t ldc, int tiles_m, int tiles_n, int splits,
                    int64_t kchunk, float* __restrict__ partials, uint32_t idesc, uint32_t* status, const ConvTma conv,
                    int out16, int seg_kblocks) {
    constexpr int STAGES = PAIR_STAGES, NACC = PAIR_NACC, BN = PAIR_BN;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    // layout (identical in both CTAs): [stages][C staging tiles of the epilogue warps][barriers]
    float* store_stage = reinterpret_cast<float*>(smem_al + STAGES * PAIR_STAGE_BYTES);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * PAIR_STAGE_BYTES + PAIR_STORE_BYTES);
    const uint32_t bar0 = smem_base + STAGES * PAIR_STAGE_BYTES + PAIR_STORE_BYTES;
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + NACC + a); };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + 2 * STAGES + 2 * NACC);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = leader
    const bool leader = rank == 0;

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 32) {      // descriptors into the TMA unit's cache while the barriers are set up
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmB);
        if (store_via_tma) prefetch_tensormap(&tmC);
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < NACC; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 2 * EPI_WARPS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {   // the same warp of both CTAs allocates: the pair's tensor memory is handed out together
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)(NACC * BN)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    cluster_sync_all();        // the peer's barriers exist before anything of this CTA can arrive on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    asm volatile("griddepcontrol.wait;" ::: "memory");

    const int64_t items = (int64_t)tiles_m * tiles_n * splits;
    const int64_t pair_id = blockIdx.x >> 1, pairs = gridDim.x >> 1;
    constexpr int GROUP = 8;     // 8 tile rows of 256 = the 2048 rows a group of the single-CTA kernel covers
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
    // seg_kblocks > 0 (fp32 data as three bfloat16 pieces each): op(A) and op(B) hold their pieces one after the other
    // along k, seg_kblocks k blocks per piece, and a tile's k loop walks six (piece of A, piece of B) segments, the
    // smallest products first, all into the same accumulator
    auto kblocks_of = [&](int sp, int64_t& kbeg) {
        if (seg_kblocks > 0) { kbeg = 0; return 6 * seg_kblocks; }
        kbeg = (int64_t)sp * kchunk;
        const int64_t kend = min(k, kbeg + kchunk);
        return (int)((kend - kbeg + TBK - 1) / TBK);
    };

    if (warp == 0) {
        // ------------------------------------------------ TMA producer (both CTAs)
        if (lane == 0) {
            uint32_t cnt = 0;
            bool ok = true;
            for (int64_t item = pair_id; item < items && ok; item += pairs) {
                int tm, tn, sp;
                decode(item, tm, tn, sp);
                int64_t kbeg;
                const int kb_n = kblocks_of(sp, kbeg);
                const int32_t m0 = tm * (2 * TBM) + (int32_t)rank * TBM;            // this CTA's rows of op(A)
                const int32_t n0 = tn * BN + (int32_t)rank * PAIR_HALF_N;           // this CTA's columns of op(B)
                int32_t cw = 0, ch = 0, cn = 0;
                if (CONV) conv_tile_origin(conv, (int64_t)tn * BN + (int64_t)rank * PAIR_HALF_N, cw, ch, cn);
                for (int kb = 0; kb < kb_n; ++kb, ++cnt) {
                    const int s = cnt % STAGES;
                    const uint32_t ph = (cnt / STAGES) & 1;
                    if (!mbar_wait(empty_bar(s), ph ^ 1, abort_flag, status,
                                   STATUS_MARK | (ROLE_TMA << 16) | (BAR_EMPTY << 8) | s)) { ok = false; break; }
                    const uint32_t sa = smem_base + s * PAIR_STAGE_BYTES;
                    const uint32_t sb = sa + PAIR_A_BYTES;
                    int32_t k0 = (int32_t)(kbeg + (int64_t)kb * TBK), k0a = k0;
                    if (seg_kblocks > 0) {
                        // segments (piece of A, piece of B): (2,0) (0,2) (1,1) (1,0) (0,1) (0,0), two bits per entry
                        const int seg = kb / seg_kblocks, kk = kb - seg * seg_kblocks;
                        k0a = (int32_t)((((0x052 >> (2 * seg)) & 3) * seg_kblocks + kk) * TBK);
                        k0 = (int32_t)((((0x118 >> (2 * seg)) & 3) * seg_kblocks + kk) * TBK);
                    }
                    if (leader) mbar_expect_tx(full_bar(s), 2 * PAIR_STAGE_BYTES);   // both CTAs' bytes
                    const uint32_t fb = map_to_cta(full_bar(s), 0);
                    if (A_MN) {
#pragma unroll
                        for (int c = 0; c < TBM / 64; ++c) tma_load_2d_pair(&tmA, sa + c * (64 * TBK * 2), fb, m0 + c * 64, k0a);
                    } else {
                        tma_load_2d_pair(&tmA, sa, fb, k0a, m0);
                    }
                    if (CONV) {
                        const int kg = k0 / TBK;
                        const int tap = kg / conv.chunks, c0 = (kg - tap * conv.chunks) * TBK;
                        const int fr = tap / conv.kw, fs = tap - fr * conv.kw;
                        tma_load_im2col_pair(&tmB, sb, fb, c0, cw, ch, cn, (uint16_t)fs, (uint16_t)fr);
                    } else if (B_MN) {
#pragma unroll
                        for (int c = 0; c < PAIR_HALF_N / 64; ++c) tma_load_2d_pair(&tmB, sb + c * (64 * TBK * 2), fb, n0 + c * 64, k0);
                    } else {
                        tma_load_2d_pair(&tmB, sb, fb, k0, n0);
                    }
                }
            }
            // drain: the leader's full barriers count the copies of both CTAs; neither CTA leaves before the
            // cluster-wide barrier below, so no copy that was armed can land in the memory of a CTA that is gone
            if (leader) {
                const uint32_t armed = cnt < (uint32_t)STAGES ? cnt : (uint32_t)STAGES;
                for (uint32_t i = 0; i < armed; ++i) {
                    const uint32_t c = cnt - 1 - i;
                    const int s = c % STAGES;
                    const uint32_t ph = (c / STAGES) & 1;
                    for (uint32_t it = 0; it < (1u << 20); ++it)
                        if (mbar_try_wait(full_bar(s), ph)) break;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (one thread of the leader CTA)
        if (leader && lane == 0) {
            uint32_t cnt = 0, it = 0;
            bool ok = true;
            for (int64_t item = pair_id; item < items && ok; item += pairs, ++it) {
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
                    const uint32_t sa = smem_base + s * PAIR_STAGE_BYTES;
                    const uint32_t sb = sa + PAIR_A_BYTES;
#pragma unroll
                    for (int kk = 0; kk < TBK / UMMA_K; ++kk) {
                        // descriptors name offsets that hold in both CTAs: each supplies its own rows of A and its
                        // own half of B's columns from the same place in its shared memory
                        const uint64_t ad = A_MN ? smem_desc(sa + kk * (UMMA_K * 128), TBK * 128, 1024)
                                                 : smem_desc(sa + kk * (UMMA_K * 2), 0, 1024);
                        const uint64_t bd = B_MN ? smem_desc(sb + kk * (UMMA_K * 128), TBK * 128, 1024)
                                                 : smem_desc(sb + kk * (UMMA_K * 2), 0, 1024);
                        umma_f16_pair(d_tmem, ad, bd, idesc, (kb | kk) != 0);
                    }
                    umma_commit_pair(empty_bar(s), 3);          // frees the stage in both CTAs
                }
                if (!ok) break;
                umma_commit_pair(tfull_bar(acc), 3);            // accumulator complete, in both CTAs
            }
        }
    } else {
        // ------------------------------------------------ epilogue (warps 2..9 of both CTAs)
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        float* stage = store_stage + (warp - 2) * (32 * 32);
        const uint32_t tempty_leader0 = map_to_cta(tempty_bar(0), 0);
        uint32_t it = 0, sbuf = 0;
        bool ok = true;
        for (int64_t item = pair_id; item < items && ok; item += pairs, ++it) {
            int tm, tn, sp;
            decode(item, tm, tn, sp);
            const uint32_t acc = it % NACC, aph = (it / NACC) & 1;
            if (!mbar_wait(tfull_bar(acc), aph, abort_flag, status,
                           STATUS_MARK | (ROLE_EPI << 16) | (BAR_TMEM_FULL << 8) | acc)) { ok = false; break; }
            tc_fence_after();
            const int64_t row0 = (int64_t)tm * (2 * TBM) + (int64_t)rank * TBM + q * 32;
            const bool raw = splits > 1;
            float* out = raw ? partials + (int64_t)sp * m * n : C;
            const bool via_tma = raw ? (store_via_tma == 2) : (store_via_tma == 1);
            auto release = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(tempty_leader0 + 8u * acc);
            };
            const uint32_t tacc = tmem_base + acc * BN + ((uint32_t)(q * 32) << 16);
            bool done = false;
            if constexpr (OUT16) {
                if (!raw) {      // 16-bit result: one rounding at the store (split-k partial sums stay fp32)
                    epilogue_tile16<BN, 1>(tacc, row0, (int64_t)tn * BN, half, lane, m, n, alpha, beta, out, ldc,
                                                store_via_tma == 1, &tmC, stage, sbuf, out16, release);
                    done = true;
                }
            }
            if (!done)
                epilogue_tile<BN, 1>(tacc, row0, (int64_t)tn * BN, half, lane, m, n, alpha, beta, out, raw ? m : ldc,
                                          raw, via_tma, &tmC, sp, stage, sbuf, release);
        }
        if (lane == 0) bulk_wait_all();
    }

    // ------------------------------------------------ teardown: every thread of both CTAs arrives here on every path
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    cluster_sync_all();        // the peer may still read this CTA's shared memory or arrive on its barriers until here
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)(NACC * BN)) : "memory");
    }
}

template <bool A_MN, bool B_MN, bool CONV, bool OUT16>
static cudaError_t launch_pair(const GemmArgs& a, KSplit ks, float* partials, gemm_config_t* cfg) {
    CUtensorMap tmA, tmB;
    bool ok = A_MN ? make_map(&tmA, a.dtype, a.A, a.m, a.k, a.lda, 64, TBK)
                   : make_map(&tmA, a.dtype, a.A, a.k, a.m, a.lda, TBK, TBM);
    if (CONV) {
        ok = ok && make_im2col_map(&tmB, a.dtype, *a.conv, a.n / ((int64_t)a.conv->ho * a.conv->wo), PAIR_HALF_N);
    } else {
        ok = ok && (B_MN ? make_map(&tmB, a.dtype, a.B, a.n, a.k, a.ldb, 64, TBK)
                         : make_map(&tmB, a.dtype, a.B, a.k, a.n, a.ldb, TBK, PAIR_HALF_N));
    }
    if (!ok) return cudaErrorInvalidValue;
    CUtensorMap tmC = tmA;
    int store_via_tma = 0;
    if (ks.splits == 1 && c_tma_addressable(a.C, a.m, a.ldc, a.out16))
        store_via_tma = make_c_map(&tmC, a.C, a.m, a.n, a.ldc, a.out16) ? 1 : 0;
    if (ks.splits > 1 && (reinterpret_cast<uintptr_t>(partials) & 15) == 0 && a.m % 4 == 0 && a.m * a.n * 4 < (1LL << 40))
        store_via_tma = make_partials_map(&tmC, partials, a.m, a.n, ks.splits) ? 2 : 0;

    static std::atomic<bool> attr_set[64];      // zero-initialised; set once per device
    auto kern = tc_gemm_pair_kernel<A_MN, B_MN, CONV, OUT16>;
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev].load()) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, PAIR_SMEM_BYTES);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev].store(true);
    }
    const int64_t tiles_m = (a.m + 2 * TBM - 1) / (2 * TBM), tiles_n = (a.n + PAIR_BN - 1) / PAIR_BN;
    if (tiles_m > 0x7FFFFFFF || tiles_n > 0x7FFFFFFF || tiles_m * tiles_n > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const int64_t items = tiles_m * tiles_n * ks.splits;
    const int64_t max_pairs = sm_count() / 2;
    const int grid = 2 * (int)(items < max_pairs ? items : max_pairs);
    cfg->tile_m = 2 * TBM; cfg->tile_n = PAIR_BN; cfg->tile_k = TBK; cfg->stages = PAIR_STAGES; cfg->grid = grid;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)grid);
    lc.blockDim = dim3(TC_THREADS);
    lc.dynamicSmemBytes = PAIR_SMEM_BYTES;
    lc.stream = a.stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 2;
    cudaError_t le = cudaLaunchKernelEx(&lc, kern, tmA, tmB, tmC, store_via_tma, a.m, a.n, a.k, a.alpha, a.beta, a.C, a.ldc,
                                        (int)tiles_m, (int)tiles_n, ks.splits, ks.chunk,
                                        ks.splits > 1 ? partials : (float*)nullptr,
                                        instr_desc(a.dtype, A_MN, B_MN, 2 * TBM, PAIR_BN), a.status, conv_tma_params(a.conv), a.out16,
                                        (int)(a.seg_k / TBK));
    return le != cudaSuccess ? le : cudaGetLastError();
}

cudaError_t launch_tensor_pair(const GemmArgs& a, KSplit ks, float* partials, gemm_config_t* cfg) {
    cfg->kernel = GEMM_KERNEL_TENSOR;
    cfg->split_k = ks.splits;
    cfg->vector_a = cfg->vector_b = 1;
    const bool a_mn = !a.ta, b_mn = a.tb;
    if (a.conv != nullptr)
        return a_mn ? (a.out16 ? launch_pair<true, false, true, true>(a, ks, partials, cfg)
                               : launch_pair<true, false, true, false>(a, ks, partials, cfg))
                    : (a.out16 ? launch_pair<false, false, true, true>(a, ks, partials, cfg)
                               : launch_pair<false, false, true, false>(a, ks, partials, cfg));
    if (a_mn && b_mn) return (a.out16 ? launch_pair<true, true, false, true>(a, ks, partials, cfg) : launch_pair<true, true, false, false>(a, ks, partials, cfg));
    if (a_mn && !b_mn) return (a.out16 ? launch_pair<true, false, false, true>(a, ks, partials, cfg) : launch_pair<true, false, false, false>(a, ks, partials, cfg));
    if (!a_mn && b_mn) return (a.out16 ? launch_pair<false, true, false, true>(a, ks, partials, cfg) : launch_pair<false, true, false, false>(a, ks, partials, cfg));
    return (a.out16 ? launch_pair<false, false, false, true>(a, ks, partials, cfg) : launch_pair<false, false, false, false>(a, ks, partials, cfg));
}

}  // namespace b200gemm
