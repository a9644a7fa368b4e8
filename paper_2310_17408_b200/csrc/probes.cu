// Peak-confirmation probes: the three rates the GEMM kernels are judged against, measured by this library's own
// code on the device it runs on.  They are the counterpart of the paper's "solo mode" (Section IV-A: the micro-kernel
// called on its own, operands resident in the fastest memory), one per unit that bounds a kernel here:
//   gemm_probe_copy   HBM: a streaming copy (bytes read + bytes written per second)
//   gemm_probe_ffma   CUDA cores: fp32 FMA loops, as independent register-only chains and as the SIMT kernel's 8 x 8
//                     micro-kernel fed from shared memory (scalar and packed fma.rn.f32x2 forms)
//   gemm_probe_umma   tensor cores: tcgen05.mma on operands that stay in shared memory, accumulators in TMEM
// Every probe has a bounded run time (iteration counts are capped), touches no caller memory except the two
// buffers handed to the copy probe, and times itself with CUDA events on the caller's stream.
#include "tc_common.cuh"

namespace b200gemm {

__device__ float g_probe_sink[32];      // results land here only under a condition that never holds

// ---------------------------------------------------------------- HBM copy

// Each block walks whole 32 KB pieces (256 threads x 8 x 16 bytes), all eight loads of a thread issued before its
// first store, so that a block keeps 32 KB in flight and touches DRAM in long contiguous runs.
constexpr int COPY_THREADS = 256, COPY_UNROLL = 8;
__global__ void __launch_bounds__(COPY_THREADS)
probe_copy_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t n) {
    constexpr size_t PIECE = (size_t)COPY_THREADS * COPY_UNROLL;
    const size_t pieces = n / PIECE;
    for (size_t p = blockIdx.x; p < pieces; p += gridDim.x) {
        const size_t base = p * PIECE + threadIdx.x;
        uint4 v[COPY_UNROLL];
#pragma unroll
        for (int u = 0; u < COPY_UNROLL; ++u) v[u] = __ldcs(src + base + (size_t)u * COPY_THREADS);
#pragma unroll
        for (int u = 0; u < COPY_UNROLL; ++u) __stcs(dst + base + (size_t)u * COPY_THREADS, v[u]);
    }
    for (size_t i = pieces * PIECE + (size_t)blockIdx.x * COPY_THREADS + threadIdx.x; i < n; i += (size_t)gridDim.x * COPY_THREADS)
        __stcs(dst + i, __ldcs(src + i));
}

// ---------------------------------------------------------------- fp32 FMA, registers only

// 16 independent dependency chains per thread: the issue-rate ceiling of the FMA pipes
__global__ void __launch_bounds__(256)
probe_ffma_chains_kernel(int iters, float x, float y) {
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = (float)(threadIdx.x + i);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = fmaf(acc[i], x, y);
    }
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) s += acc[i];
    if (s == 1.2345678e-30f) g_probe_sink[threadIdx.x & 31] = s;
}

// The micro-kernel of a GEMM thread on its own: an 8 x 8 block of accumulators receives one outer product a (8) x b (8)
// per k, a and b read from shared memory with two 128-bit loads each, as the SIMT kernel's threads read their
// fragments (one slice of 8 k per loop trip, the next k's fragments loaded while the current ones are used); no global
// traffic, no stores, no barriers inside the loop.  PACKED: two FMAs per fma.rn.f32x2, accumulators held as pairs of
// neighbouring columns and every a duplicated into a pair, the arrangement of the SIMT kernel; otherwise scalar FMAs,
// row by row with the columns there and back.
constexpr int PROBE_BK = 8, PROBE_LD = 132;       // rows of 128 floats + 4 of padding, as the kernel's stages
template <bool PACKED>
__global__ void __launch_bounds__(256, 2)
probe_ffma_block_kernel(int iters, float x) {
    __shared__ __align__(16) float As[PROBE_BK * PROBE_LD];
    __shared__ __align__(16) float Bs[PROBE_BK * PROBE_LD];
    for (int i = threadIdx.x; i < PROBE_BK * PROBE_LD; i += 256) {
        As[i] = x * (float)(i % 7);
        Bs[i] = x * (float)(i % 5);
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // fragment offsets: 0..28 (+32) of a row of A, 0..76 (+16) of a row of B: inside the 128 floats of a row
    const float* ap = As + (lane & 7) * 4;
    const float* bp = Bs + (lane >> 3) * 4 + (warp & 1) * 64;
    float s = 0.0f;
    if (!PACKED) {
        float acc[8][8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[j][i] = 0.0f;
        for (int it = 0; it < iters; ++it) {
            float a[2][8], b[2][8];
            auto frag = [&](int kk, int buf) {
                const float4 a0 = *reinterpret_cast<const float4*>(ap + kk * PROBE_LD);
                const float4 a1 = *reinterpret_cast<const float4*>(ap + kk * PROBE_LD + 32);
                const float4 b0 = *reinterpret_cast<const float4*>(bp + kk * PROBE_LD);
                const float4 b1 = *reinterpret_cast<const float4*>(bp + kk * PROBE_LD + 16);
                a[buf][0] = a0.x; a[buf][1] = a0.y; a[buf][2] = a0.z; a[buf][3] = a0.w;
                a[buf][4] = a1.x; a[buf][5] = a1.y; a[buf][6] = a1.z; a[buf][7] = a1.w;
                b[buf][0] = b0.x; b[buf][1] = b0.y; b[buf][2] = b0.z; b[buf][3] = b0.w;
                b[buf][4] = b1.x; b[buf][5] = b1.y; b[buf][6] = b1.z; b[buf][7] = b1.w;
            };
            frag(0, 0);
#pragma unroll
            for (int kk = 0; kk < PROBE_BK; ++kk) {
                if (kk + 1 < PROBE_BK) frag(kk + 1, (kk + 1) & 1);
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) {
                        const int j = (i & 1) ? 7 - jj : jj;
                        acc[j][i] = fmaf(a[kk & 1][i], b[kk & 1][j], acc[j][i]);
                    }
            }
            asm volatile("" ::: "memory");      // the next trip reads its fragments again
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int i = 0; i < 8; ++i) s += acc[j][i];
    } else {
        uint64_t P[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) P[i][j] = 0ull;
        auto pack = [](float lo, float hi) { uint64_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r; };
        for (int it = 0; it < iters; ++it) {
            uint64_t a[2][8], b[2][4];
            auto frag = [&](int kk, int buf) {
                const float4 a0 = *reinterpret_cast<const float4*>(ap + kk * PROBE_LD);
                const float4 a1 = *reinterpret_cast<const float4*>(ap + kk * PROBE_LD + 32);
                const float4 b0 = *reinterpret_cast<const float4*>(bp + kk * PROBE_LD);
                const float4 b1 = *reinterpret_cast<const float4*>(bp + kk * PROBE_LD + 16);
                b[buf][0] = pack(b0.x, b0.y); b[buf][1] = pack(b0.z, b0.w);
                b[buf][2] = pack(b1.x, b1.y); b[buf][3] = pack(b1.z, b1.w);
                a[buf][0] = pack(a0.x, a0.x); a[buf][1] = pack(a0.y, a0.y);
                a[buf][2] = pack(a0.z, a0.z); a[buf][3] = pack(a0.w, a0.w);
                a[buf][4] = pack(a1.x, a1.x); a[buf][5] = pack(a1.y, a1.y);
                a[buf][6] = pack(a1.z, a1.z); a[buf][7] = pack(a1.w, a1.w);
            };
            frag(0, 0);
#pragma unroll
            for (int kk = 0; kk < PROBE_BK; ++kk) {
                if (kk + 1 < PROBE_BK) frag(kk + 1, (kk + 1) & 1);
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(P[i][j]) : "l"(a[kk & 1][i]), "l"(b[kk & 1][j]));
            }
            asm volatile("" ::: "memory");
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float lo, hi;
                asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(P[i][j]));
                s += lo + hi;
            }
    }
    if (s == 1.2345678e-30f) g_probe_sink[threadIdx.x & 31] = s;
}

// ---------------------------------------------------------------- tcgen05.mma on shared-memory-resident operands

constexpr int PROBE_RING = 6;           // k blocks in flight between issue and completion, as in the GEMM pipelines
constexpr int PROBE_N = 256;
constexpr int PROBE_A_BYTES = TBM * TBK * 2;

// One CTA per SM (PAIR: one cluster of two CTAs per SM pair).  The operand tiles (A 128 x 64, B 256 x 64 — PAIR: each
// CTA half of B's rows — 16-bit, K-major, 128-byte swizzle atoms) are written once by plain stores and then read by
// every MMA; no TMA, no global memory traffic.  One thread issues k blocks of four 128(256) x 256 x 16 MMAs, commits
// each block to a ring of mbarriers and waits (bounded) for the block issued PROBE_RING earlier.
template <bool PAIR>
__global__ void __launch_bounds__(128, 1)
probe_umma_kernel(int kblocks, uint32_t idesc, uint32_t* status, int f16) {
    constexpr int B_BYTES = (PAIR ? PROBE_N / 2 : PROBE_N) * TBK * 2;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + PROBE_A_BYTES + B_BYTES);
    const uint32_t bar0 = smem_base + PROBE_A_BYTES + B_BYTES;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bars + PROBE_RING);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool leader = !PAIR || cluster_ctarank() == 0;

    if (threadIdx.x == 0) {
        for (int r = 0; r < PROBE_RING; ++r) mbar_init(bar0 + 8u * r, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {      // a whole, converged warp allocates tensor memory (warp 0 is busy with the barriers)
        if (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)PROBE_N) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                         ::"r"(smem_u32((const void*)tmem_slot)), "r"((uint32_t)PROBE_N) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    // operand values: a fixed pattern of small finite numbers (any bits that are not NaN / Inf would do; real
    // values keep the multipliers' switching activity, and with it power and clocks, like a GEMM's)
    {
        uint16_t* ops = reinterpret_cast<uint16_t*>(smem_al);
        for (int i = threadIdx.x; i < (PROBE_A_BYTES + B_BYTES) / 2; i += blockDim.x) {
            uint32_t h = (uint32_t)i * 2654435761u + blockIdx.x * 40503u;
            h ^= h >> 15;
            const float v = (float)((int)(h & 0xFF) - 128) * (1.0f / 256.0f);
            ops[i] = f16 ? __half_as_ushort(__float2half_rn(v)) : __bfloat16_as_ushort(__float2bfloat16_rn(v));
        }
        fence_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) { __syncwarp(); cluster_sync_all(); }
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0 && lane == 0 && leader) {
        const uint32_t sa = smem_base, sb = smem_base + PROBE_A_BYTES;
        bool ok = true;
        for (int kb = 0; kb < kblocks && ok; ++kb) {
            const int r = kb % PROBE_RING;
            if (kb >= PROBE_RING) {
                ok = mbar_wait(bar0 + 8u * r, (uint32_t)(kb / PROBE_RING - 1) & 1u, abort_flag, status,
                               STATUS_MARK | (ROLE_SELFTEST << 16) | (BAR_EMPTY << 8) | r);
                if (!ok) break;
                tc_fence_after();
            }
#pragma unroll
            for (int kk = 0; kk < TBK / UMMA_K; ++kk) {
                const uint64_t ad = smem_desc(sa + kk * (UMMA_K * 2), 0, 1024);
                const uint64_t bd = smem_desc(sb + kk * (UMMA_K * 2), 0, 1024);
                if (PAIR) umma_f16_pair(tmem_base, ad, bd, idesc, (kb | kk) != 0);
                else umma_f16(tmem_base, ad, bd, idesc, (kb | kk) != 0);
            }
            if (PAIR) umma_commit_pair(bar0 + 8u * r, 1);      // arrives in the leader only
            else umma_commit(bar0 + 8u * r);
        }
        // completion of everything still in flight (each barrier's last use)
        const int tail = kblocks < PROBE_RING ? kblocks : PROBE_RING;
        for (int i = 0; i < tail && ok; ++i) {
            const int kb = kblocks - 1 - i;
            ok = mbar_wait(bar0 + 8u * (kb % PROBE_RING), (uint32_t)(kb / PROBE_RING) & 1u, abort_flag, status,
                           STATUS_MARK | (ROLE_SELFTEST << 16) | (BAR_FULL << 8) | (kb % PROBE_RING));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) { __syncwarp(); cluster_sync_all(); }     // the peer's shared memory is read by the pair's MMAs until here
    if (warp == 1) {
        tc_fence_after();
        if (PAIR)
            asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)PROBE_N) : "memory");
        else
            asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)PROBE_N) : "memory");
    }
}

// runs `launch` once untimed and once between two events on `s`; returns the timed duration
template <typename F>
static cudaError_t timed(cudaStream_t s, F&& launch, double* ms_out) {
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    if (e == cudaSuccess) e = launch();
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e == cudaSuccess) e = cudaEventRecord(e0, s);
    if (e == cudaSuccess) e = launch();
    if (e == cudaSuccess) e = cudaEventRecord(e1, s);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    float ms = 0.0f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    *ms_out = (double)ms;
    return e;
}

}  // namespace b200gemm

using namespace b200gemm;

extern "C" {

int gemm_probe_copy(void* dst, const void* src, size_t bytes, double* gbs, double* ms, void* stream) {
    if (dst == nullptr || (reinterpret_cast<uintptr_t>(dst) & 15)) return -1;
    if (src == nullptr || (reinterpret_cast<uintptr_t>(src) & 15)) return -2;
    if (bytes < 16 || bytes % 16 != 0 || bytes > ((size_t)64 << 30)) return -3;
    if (gbs == nullptr) return -4;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t n = bytes / 16;
    const int blocks = sm_count() * 8;
    double t = 0.0;
    const cudaError_t e = timed(s, [&]() {
        probe_copy_kernel<<<blocks, COPY_THREADS, 0, s>>>(static_cast<const uint4*>(src), static_cast<uint4*>(dst), n);
        return cudaGetLastError();
    }, &t);
    if (e != cudaSuccess) { note_launch_error(e); return GEMM_ERR_LAUNCH; }
    *gbs = t > 0.0 ? 2.0 * (double)bytes / (t * 1e-3) / 1e9 : 0.0;
    if (ms) *ms = t;
    return GEMM_OK;
}

int gemm_probe_ffma(int pattern, int iters, double* tflops, double* ms, void* stream) {
    if (pattern < 0 || pattern > 2) return -1;
    if (iters < 1 || iters > (1 << 16)) return -2;
    if (tflops == nullptr) return -3;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int sms = sm_count();
    double t = 0.0, flops = 0.0;
    cudaError_t e;
    if (pattern == 0) {
        const int blocks = sms * 8;       // 2048 threads per SM
        flops = (double)blocks * 256.0 * iters * 8.0 * 16.0 * 2.0;
        e = timed(s, [&]() { probe_ffma_chains_kernel<<<blocks, 256, 0, s>>>(iters, 0.999f, 0.001f); return cudaGetLastError(); }, &t);
    } else {
        const int blocks = sms * 2;       // the SIMT kernel's residency: two 256-thread CTAs per SM
        flops = (double)blocks * 256.0 * iters * 8.0 * 64.0 * 2.0;
        e = timed(s, [&]() {
            if (pattern == 1) probe_ffma_block_kernel<false><<<blocks, 256, 0, s>>>(iters, 1e-3f);
            else probe_ffma_block_kernel<true><<<blocks, 256, 0, s>>>(iters, 1e-3f);
            return cudaGetLastError();
        }, &t);
    }
    if (e != cudaSuccess) { note_launch_error(e); return GEMM_ERR_LAUNCH; }
    *tflops = t > 0.0 ? flops / (t * 1e-3) / 1e12 : 0.0;
    if (ms) *ms = t;
    return GEMM_OK;
}

int gemm_probe_umma(int dtype, int pair, int kblocks, double* tflops, double* ms, void* stream) {
    if (dtype != GEMM_F16 && dtype != GEMM_BF16) return -1;
    if (pair != 0 && pair != 1) return -2;
    if (kblocks < 1 || kblocks > (1 << 18)) return -3;
    if (tflops == nullptr) return -4;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t* status = nullptr;
    bool arch_ok = false;
    if (!device_info(&status, &arch_ok)) return GEMM_ERR_LAUNCH;
    if (!arch_ok) return GEMM_ERR_ARCH;
    const int sms = sm_count();
    const int smem = PROBE_A_BYTES + (pair ? PROBE_N / 2 : PROBE_N) * TBK * 2 + 1024 + 256;
    cudaError_t e = pair ? cudaFuncSetAttribute(probe_umma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
                         : cudaFuncSetAttribute(probe_umma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) { note_launch_error(e); return GEMM_ERR_LAUNCH; }
    const int grid = pair ? (sms / 2) * 2 : sms;
    const int mma_m = pair ? 2 * TBM : TBM;
    const uint32_t idesc = instr_desc(dtype, false, false, mma_m, PROBE_N);
    const double flops = (double)(pair ? grid / 2 : grid) * kblocks * 2.0 * mma_m * PROBE_N * TBK;
    double t = 0.0;
    e = timed(s, [&]() {
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3((unsigned)grid);
        lc.blockDim = dim3(128);
        lc.dynamicSmemBytes = smem;
        lc.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = pair ? 2 : 1;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        lc.attrs = attr;
        lc.numAttrs = 1;
        cudaError_t le = pair ? cudaLaunchKernelEx(&lc, probe_umma_kernel<true>, kblocks, idesc, status, dtype == GEMM_F16 ? 1 : 0)
                              : cudaLaunchKernelEx(&lc, probe_umma_kernel<false>, kblocks, idesc, status, dtype == GEMM_F16 ? 1 : 0);
        return le != cudaSuccess ? le : cudaGetLastError();
    }, &t);
    if (e != cudaSuccess) { note_launch_error(e); return GEMM_ERR_LAUNCH; }
    *tflops = t > 0.0 ? flops / (t * 1e-3) / 1e12 : 0.0;
    if (ms) *ms = t;
    return GEMM_OK;
}

}  // extern "C"
