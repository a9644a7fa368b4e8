// Device-side building blocks shared by the tcgen05 kernels: bounded mbarrier waits, TMA copies, shared-memory
// matrix descriptors, MMA issue / commit, TMEM loads; and the host-side tensor-map builders.
#pragma once
#include <cuda.h>

#include "internal.cuh"

namespace b200gemm {

constexpr int TBM = 128;            // MMA M (TMEM lanes)
constexpr int TBK = 64;             // k block: 64 x 2 bytes = one 128-byte swizzle row
constexpr int UMMA_K = 16;          // k extent of one tcgen05.mma for 16-bit inputs
constexpr int EPI_WARPS = 8;        // two epilogue warps per TMEM lane quarter, each taking every other 32-column chunk
constexpr int TC_THREADS = 64 + 32 * EPI_WARPS;
constexpr uint32_t SPIN_FAST = 4096;
constexpr uint32_t SPIN_LIMIT = 1u << 24;   // then ~128 ns sleeps: gives up after a few seconds

enum Role : uint32_t { ROLE_TMA = 1, ROLE_MMA = 2, ROLE_EPI = 3, ROLE_SELFTEST = 0x7F };
enum Bar : uint32_t { BAR_FULL = 1, BAR_EMPTY = 2, BAR_TMEM_FULL = 3, BAR_TMEM_EMPTY = 4 };

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false if the wait expired or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* status, uint32_t code, uint32_t limit = SPIN_LIMIT) {
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it >= SPIN_FAST) {
            if (*abort_flag) return false;
            __nanosleep(128);
        }
    }
    atomicCAS(status, 0u, code);
    *abort_flag = 1;
    return false;
}

// brings a tensor map (a kernel parameter) into the TMA unit's descriptor cache ahead of its first use
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tm) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

__device__ __forceinline__ void tma_load_2d(const CUtensorMap* tm, uint32_t dst, uint32_t bar, int32_t c0, int32_t c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1) : "memory");
}

// the same from a 3-D map (a strided batch of matrices: the third coordinate is the problem index, the box one deep)
__device__ __forceinline__ void tma_load_3d(const CUtensorMap* tm, uint32_t dst, uint32_t bar, int32_t c0, int32_t c1, int32_t c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// TMA load in im2col mode from an NHWC tensor (tensor map dimensions C, W, H, N): the box holds `pixelsPerColumn`
// consecutive output pixels starting at the one whose receptive field begins at (w, h) of image n, each with
// `channelsPerPixel` channels from c on, read at filter-tap offset (off_w, off_h); positions outside the image are
// zero-filled.  Rows of the box are pixels, so the stage is the K-major operand tile of the lowered matrix.
__device__ __forceinline__ void tma_load_im2col(const CUtensorMap* tm, uint32_t dst, uint32_t bar, int32_t c, int32_t w,
                                                int32_t h, int32_t n, uint16_t off_w, uint16_t off_h) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
        ::"r"(dst), "l"(tm), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h) : "memory");
}

// geometry the producer needs to turn (tile column, k block) into im2col coordinates
struct ConvTma {
    int32_t ho, wo;        // output extent
    int32_t stride, pad;   // same in both directions
    int32_t kw;            // filter width
    int32_t chunks;        // C_in / 64: k blocks per filter tap
};
// first pixel j of a tile -> tensor coordinates of its receptive field's corner
__device__ __forceinline__ void conv_tile_origin(const ConvTma& cv, int64_t j, int32_t& w, int32_t& h, int32_t& n) {
    const int hw = cv.ho * cv.wo;
    n = (int32_t)(j / hw);
    const int rem = (int)(j - (int64_t)n * hw);
    const int oh = rem / cv.wo, ow = rem - oh * cv.wo;
    w = ow * cv.stride - cv.pad;
    h = oh * cv.stride - cv.pad;
}

// shared memory -> global tile store (bulk async group); out-of-range parts of the box are clipped by the hardware
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, uint32_t src, int32_t c0, int32_t c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(tm), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tm, uint32_t src, int32_t c0, int32_t c1, int32_t c2) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(tm), "r"(src), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// shared-memory matrix descriptor (128-byte swizzle): start address, leading / stride byte offsets in 16-byte units
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;      // descriptor version of the tcgen05 family
    d |= (uint64_t)2 << 61;      // swizzle mode: 128 bytes
    return d;
}

__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives on the mbarrier once all previously issued MMAs of this thread have completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
// 32 columns of a binary16 accumulator (one 16-bit value in the low half of each 32-bit TMEM column), two columns
// packed into each of 16 registers: low half = even column, high half = odd column
__device__ __forceinline__ void tmem_ld16_packed(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.pack::16b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- CTA pairs (clusters of two CTAs, tcgen05 cta_group::2)
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster (shared::cluster window)
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load of a CTA pair: destination in the executing CTA, completion on an mbarrier given by its cluster address
__device__ __forceinline__ void tma_load_2d_pair(const CUtensorMap* tm, uint32_t dst, uint32_t bar_cluster, int32_t c0, int32_t c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tm), "r"(bar_cluster), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_im2col_pair(const CUtensorMap* tm, uint32_t dst, uint32_t bar_cluster, int32_t c,
                                                     int32_t w, int32_t h, int32_t n, uint16_t off_w, uint16_t off_h) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2], {%7, %8};"
        ::"r"(dst), "l"(tm), "r"(bar_cluster), "r"(c), "r"(w), "r"(h), "r"(n), "h"(off_w), "h"(off_h) : "memory");
}
__device__ __forceinline__ void umma_f16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives, in every CTA of `mask`, on the mbarrier at this shared-memory offset once the pair's MMAs issued so far
// have completed
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint16_t mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}

// Epilogue of one accumulator tile for one warp (lane = row of C, TMEM lanes 32q .. 32q+31 starting at row0).
// The warp takes the 32-column chunks half, half + 2, ... of the BN-wide tile: each chunk is read from TMEM, scaled
// (alpha, beta of Fig. 3; raw = split-k partial sums, stored unscaled) and then either written straight to global
// memory (32 consecutive floats of one column per instruction) or, when the target can be addressed by TMA,
// transposed through a 32 x 32 staging tile in shared memory and written by an asynchronous bulk tensor store,
// which also clips the tile at the matrix edge.  release_acc() is called exactly once, as soon as the warp has
// read its last chunk, so that the accumulator can be overwritten while the stores are still in flight.
template <int BN, int STORE_BUFS, typename Release>
__device__ __forceinline__ void epilogue_tile(uint32_t tmem_acc, int64_t row0, int64_t n0, int half, int lane,
                                              int64_t m, int64_t n, float alpha, float beta, float* out, int64_t ldo,
                                              bool raw, bool via_tma, const CUtensorMap* tmC, int sp, float* stage,
                                              uint32_t& sbuf, Release&& release_acc) {
    const int64_t row = row0 + lane;
    bool released = false;
    if (row0 < m) {
#pragma unroll 1
        for (int c = half; c < BN / 32; c += 2) {
            const int64_t col0 = n0 + c * 32;
            if (col0 >= n) break;
            const bool last_chunk = (c + 2 >= BN / 32) || (col0 + 64 >= n);
            uint32_t v[32];
            tmem_ld32(tmem_acc + c * 32, v);
            float* cp = out + row + col0 * ldo;
            float c0[32];
            const bool need_c0 = !raw && beta != 0.0f;
            if (need_c0) {      // issue all reads of C before waiting on anything
#pragma unroll
                for (int j = 0; j < 32; ++j) c0[j] = (row < m && col0 + j < n) ? cp[j * ldo] : 0.0f;
            }
            tmem_ld_wait();
            if (last_chunk) { release_acc(); released = true; }
            float* r = reinterpret_cast<float*>(v);       // scaled in place
            if (!raw && (alpha != 1.0f || need_c0)) {      // alpha == 1, beta == 0: nothing to do (x * 1 is x exactly)
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    r[j] *= alpha;
                    if (need_c0) r[j] = fmaf(beta, c0[j], r[j]);
                }
            }
            if (via_tma) {
                if (lane == 0) bulk_wait_read<STORE_BUFS - 1>();   // the store that last used this staging tile has read it
                __syncwarp();
                float* st = stage + sbuf * (32 * 32);
#pragma unroll
                for (int j = 0; j < 32; ++j) st[j * 32 + lane] = r[j];
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (raw) tma_store_3d(tmC, smem_u32(st), (int32_t)row0, (int32_t)col0, sp);
                    else tma_store_2d(tmC, smem_u32(st), (int32_t)row0, (int32_t)col0);
                    bulk_commit();
                }
                sbuf = (sbuf + 1 == (uint32_t)STORE_BUFS) ? 0 : sbuf + 1;
            } else if (row < m) {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (col0 + j < n) cp[j * ldo] = r[j];
            }
        }
    }
    if (!released) release_acc();
}

// The epilogue when the roles of the operands were exchanged (C^T = op(B)^T op(A)^T is what the kernel computes: its
// rows are the columns of the caller's C).  Lane = tile row = one column of C, so the 32 tile columns of a chunk are 32
// consecutive floats of that column: each lane scales and stores them itself, four at a time, without staging.
// `m`, `n` are the kernel's extents (rows = columns of C); element (row, col) of the tile lives at out[col + row*ldo].
template <int BN, int STORE_BUFS, typename Release>
__device__ __forceinline__ void epilogue_tile_ct(uint32_t tmem_acc, int64_t row0, int64_t n0, int half, int lane,
                                                 int64_t m, int64_t n, float alpha, float beta, float* out, int64_t ldo,
                                                 bool via_tma, const CUtensorMap* tmC, float* stage, uint32_t& sbuf,
                                                 Release&& release_acc) {
    const int64_t row = row0 + lane;
    bool released = false;
    if (row0 < m) {
        const bool vec = (reinterpret_cast<uintptr_t>(out) & 15) == 0 && ldo % 4 == 0;
#pragma unroll 1
        for (int c = half; c < BN / 32; c += 2) {
            const int64_t col0 = n0 + c * 32;
            if (col0 >= n) break;
            const bool last_chunk = (c + 2 >= BN / 32) || (col0 + 64 >= n);
            uint32_t v[32];
            tmem_ld32(tmem_acc + c * 32, v);
            tmem_ld_wait();
            if (last_chunk) { release_acc(); released = true; }
            float* r = reinterpret_cast<float*>(v);
            float* cp = out + col0 + row * ldo;
            if (alpha != 1.0f || beta != 0.0f) {
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    r[j] *= alpha; r[j + 1] *= alpha; r[j + 2] *= alpha; r[j + 3] *= alpha;
                    if (beta != 0.0f && row < m) {
                        if (vec && col0 + j + 4 <= n) {
                            const float4 c0 = *reinterpret_cast<const float4*>(cp + j);
                            r[j] = fmaf(beta, c0.x, r[j]); r[j + 1] = fmaf(beta, c0.y, r[j + 1]);
                            r[j + 2] = fmaf(beta, c0.z, r[j + 2]); r[j + 3] = fmaf(beta, c0.w, r[j + 3]);
                        } else {
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                if (col0 + j + u < n) r[j + u] = fmaf(beta, cp[j + u], r[j + u]);
                        }
                    }
                }
            }
            if (via_tma) {
                // staging tile [32 tile rows][32 floats] in the 128-byte-swizzled layout the store's tensor map names:
                // 16-byte chunk q of row l sits at chunk position q ^ (l % 8), which also spreads a warp's 16-byte
                // stores over all banks; the bulk store writes 32 columns of C x 32 floats and clips at the edges
                if (lane == 0) bulk_wait_read<STORE_BUFS - 1>();
                __syncwarp();
                uint8_t* st = reinterpret_cast<uint8_t*>(stage + sbuf * (32 * 32));
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    *reinterpret_cast<float4*>(st + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                        make_float4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(tmC, smem_u32(st), (int32_t)col0, (int32_t)row0);
                    bulk_commit();
                }
                sbuf = (sbuf + 1 == (uint32_t)STORE_BUFS) ? 0 : sbuf + 1;
            } else if (row < m) {
                if (vec && col0 + 32 <= n) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<float4*>(cp + j) = make_float4(r[j], r[j + 1], r[j + 2], r[j + 3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (col0 + j < n) cp[j] = r[j];
                }
            }
        }
    }
    if (!released) release_acc();
}

// The same for a 16-bit result (out16 = GEMM_F16 or GEMM_BF16; never for split-k partial sums): `out` and tmC are
// in that type and alpha*acc + beta*C0 is rounded once, to nearest even, at the store.  Two rows of one column are
// packed into a 32-bit word before they go to the staging tile: every lane converts its values of a column pair
// (j, j+1) into one packed word, neighbouring lanes exchange these words, and a byte permute leaves the even lane with
// rows (2i, 2i+1) of column j and the odd lane with those of column j+1 (per two entries: one packed conversion,
// one shuffle, one permute, one shared-memory store).
// ACC16: the accumulator itself is binary16 (tcgen05.mma with a binary16 D): its values are widened to fp32 for the scaling.
template <int BN, int STORE_BUFS, bool ACC16 = false, typename Release>
__device__ __forceinline__ void epilogue_tile16(uint32_t tmem_acc, int64_t row0, int64_t n0, int half, int lane,
                                                int64_t m, int64_t n, float alpha, float beta, float* out, int64_t ldo,
                                                bool via_tma, const CUtensorMap* tmC, float* stage, uint32_t& sbuf,
                                                int out16, Release&& release_acc) {
    const int64_t row = row0 + lane;
    const bool odd = lane & 1;
    bool released = false;
    if (row0 < m) {
#pragma unroll 1
        for (int c = half; c < BN / 32; c += 2) {
            const int64_t col0 = n0 + c * 32;
            if (col0 >= n) break;
            const bool last_chunk = (c + 2 >= BN / 32) || (col0 + 64 >= n);
            uint32_t v[32];
            const int64_t e0 = row + col0 * ldo;
            if (ACC16) {
                uint32_t h[16];
                tmem_ld16_packed(tmem_acc + c * 32, h);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h[j]));
                    v[2 * j] = __float_as_uint(f.x);
                    v[2 * j + 1] = __float_as_uint(f.y);
                }
            } else {
                tmem_ld32(tmem_acc + c * 32, v);
                tmem_ld_wait();
            }
            if (last_chunk) { release_acc(); released = true; }
            float* r = reinterpret_cast<float*>(v);       // scaled in place
            if (alpha != 1.0f || beta != 0.0f) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    r[j] *= alpha;
                    if (beta != 0.0f && row < m && col0 + j < n) r[j] = fmaf(beta, load_c(out, out16, e0 + j * ldo), r[j]);
                }
            }
            if (via_tma) {
                if (lane == 0) bulk_wait_read<STORE_BUFS - 1>();   // the store that last used this staging tile has read it
                __syncwarp();
                uint32_t* st32 = reinterpret_cast<uint32_t*>(stage + sbuf * (32 * 32));      // [column][16 row pairs]
                // own = (column j, column j+1) of this lane's row as one packed word; the partner lane's word holds the
                // same columns of the neighbouring row; a byte permute picks (row 2i, row 2i+1) of this lane's column
                const uint32_t pick = odd ? 0x3276u : 0x5410u;
                uint32_t* dst = st32 + (odd ? 16 : 0) + (lane >> 1);
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    uint32_t own;
                    if (out16 == GEMM_F16) {
                        const __half2 h = __floats2half2_rn(r[j], r[j + 1]);
                        own = *reinterpret_cast<const uint32_t*>(&h);
                    } else {
                        const __nv_bfloat162 h = __floats2bfloat162_rn(r[j], r[j + 1]);
                        own = *reinterpret_cast<const uint32_t*>(&h);
                    }
                    const uint32_t got = __shfl_xor_sync(0xFFFFFFFFu, own, 1);
                    dst[j * 16] = __byte_perm(own, got, pick);
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    tma_store_2d(tmC, smem_u32(st32), (int32_t)row0, (int32_t)col0);
                    bulk_commit();
                }
                sbuf = (sbuf + 1 == (uint32_t)STORE_BUFS) ? 0 : sbuf + 1;
            } else if (row < m) {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                    if (col0 + j < n) store_c(out, out16, e0 + j * ldo, r[j]);
            }
        }
    }
    if (!released) release_acc();
}

// ---------------------------------------------------------------- host side (defined in tc_gemm.cu)

// 2-D map over a stored column-major matrix of 16-bit elements: dim0 = contiguous dimension (rows), dim1 = columns
// (stride ld); 128-byte swizzle
bool make_map(CUtensorMap* tm, int dtype, const void* base, int64_t rows, int64_t cols, int64_t ld,
              uint32_t box_rows, uint32_t box_cols);
// map over a strided batch of such operands: dim2 = problem index, `stride` elements apart (a multiple of 8), box one deep
bool make_map_batched(CUtensorMap* tm, int dtype, const void* base, int64_t rows, int64_t cols, int64_t ld, int64_t stride,
                      int64_t batch, uint32_t box_rows, uint32_t box_cols);
// map over the split-k partial sums [split][n][m] (fp32, dense): 32 x 32 x 1 boxes
bool make_partials_map(CUtensorMap* tm, const float* base, int64_t m, int64_t n, int splits);
// map over the result (fp32, or the 16-bit type out16) for the epilogue's tile stores: 32 x 32 boxes, no swizzle
bool make_c_map(CUtensorMap* tm, const float* base, int64_t m, int64_t n, int64_t ldc, int out16);
// map over an fp32 C for the tile stores of the exchanged-roles epilogue: dim0 = rows of C (contiguous), dim1 = columns
// (stride ldc), boxes of 32 x 32 in the 128-byte-swizzled shared-memory layout
bool make_ct_map(CUtensorMap* tm, const float* base, int64_t c_rows, int64_t c_cols, int64_t ldc);
// whether C (of either element size) can be written by TMA tile stores: 16-byte aligned base and column stride, and
// columns whose m elements end on a 16-byte boundary.  The last condition keeps the rows m..ldc-1 untouched: a tile
// store that is clipped at the matrix edge was seen to write the whole 16-byte unit the edge falls into (binary16
// result, m = 5, ldc = 8: rows 5..7 came back as zeros).
inline bool c_tma_addressable(const float* C, int64_t m, int64_t ldc, int out16) {
    const int es = out16 ? 2 : 4;
    return (reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc * es) % 16 == 0 && ldc * es < (1LL << 40) && (m * es) % 16 == 0;
}
// im2col-mode map over NHWC activations of a 16-bit type: boxes of `pixels` output pixels x 64 channels, 128-byte
// swizzle; square filter ksize, the same stride and padding in both directions
bool make_im2col_map(CUtensorMap* tm, int dtype, const ConvIndex& cv, int64_t batch, uint32_t pixels);
inline ConvTma conv_tma_params(const ConvIndex* cv) {
    if (!cv) return ConvTma{1, 1, 1, 0, 1, 1};
    return ConvTma{cv->ho, cv->wo, cv->sh, cv->ph, cv->kw, (int32_t)(cv->c_in / 64)};
}
// instruction descriptor of tcgen05.mma kind::f16: mma_m x mma_n, operand majorness, fp32 (or binary16) accumulator
uint32_t instr_desc(int dtype, bool a_mn, bool b_mn, int mma_m, int mma_n, bool acc16 = false);

}  // namespace b200gemm
