// gemm_f32_splitk_static: split-k fp32 GEMM whose partial sums live in a fixed device array that is part of
// the library image, so that the call allocates nothing.  The contract is in include/b200_gemm.h.
#include <mutex>

#include "internal.cuh"

namespace b200gemm {

// The scratch itself.  In host code the name `g_static_scratch` is only a handle for the runtime's symbol
// calls, never an address a kernel may use; the device address comes from cudaGetSymbolAddress, per device.
static __device__ __align__(256) float g_static_scratch[GEMM_STATIC_SCRATCH_BYTES / sizeof(float)];

constexpr int STATIC_MAX_DEVICES = 64;
static float* g_scratch_addr[STATIC_MAX_DEVICES];   // device address of the array on each device (nullptr = not looked up yet)
static std::mutex g_scratch_mutex;

// Set-up, once per device, with that device current: resolve the array's device address.
static cudaError_t scratch_address(float** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        float* ptr = nullptr;
        e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (ptr == nullptr) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

static bool trans_flag(char c, bool* t) {
    switch (c) {
        case 'N': case 'n': *t = false; return true;
        case 'T': case 't': case 'C': case 'c': *t = true; return true;
        default: return false;
    }
}

}  // namespace b200gemm

using namespace b200gemm;

extern "C" int gemm_f32_splitk_static(char transA, char transB, int64_t m, int64_t n, int64_t k, float alpha,
                                      const float* A, int64_t lda, const float* B, int64_t ldb, float beta, float* C,
                                      int64_t ldc, int split_k, void* stream) {
    bool ta = false, tb = false;
    if (!trans_flag(transA, &ta)) return -1;
    if (!trans_flag(transB, &tb)) return -2;
    if (m < 0) return -3;
    if (n < 0) return -4;
    if (k < 1) return -5;
    const int64_t a_rows = ta ? k : m, b_rows = tb ? n : k;
    const bool needs_ab = m > 0 && n > 0 && alpha != 0.0f;      // alpha == 0: A and B are not read and may be NULL
    if ((needs_ab && A == nullptr) || (reinterpret_cast<uintptr_t>(A) & 3)) return -7;
    if (lda < (a_rows > 1 ? a_rows : 1)) return -8;
    if ((needs_ab && B == nullptr) || (reinterpret_cast<uintptr_t>(B) & 3)) return -9;
    if (ldb < (b_rows > 1 ? b_rows : 1)) return -10;
    if (m > 0 && n > 0 && (C == nullptr || (reinterpret_cast<uintptr_t>(C) & 3))) return -12;
    if (ldc < (m > 1 ? m : 1)) return -13;
    if (split_k < 2 || split_k > 64) return -14;
    if (m == 0 || n == 0) return GEMM_OK;

    uint32_t* status = nullptr;
    bool arch_ok = false;
    if (!device_info(&status, &arch_ok)) return GEMM_ERR_LAUNCH;
    if (!arch_ok) return GEMM_ERR_ARCH;

    gemm_config_t cfg{};
    cfg.split_k = 1;
    if (alpha == 0.0f) {      // as gemm(): C <- beta*C exactly, whatever A and B hold (NaN, Inf) or point to
        GemmArgs sc{GEMM_F32, ta, tb, m, n, k, alpha, beta, A, B, C, lda, ldb, ldc, static_cast<cudaStream_t>(stream), status};
        cfg.kernel = GEMM_KERNEL_SCALE_ONLY;
        cfg.launches = beta == 1.0f ? 0 : 1;
        const cudaError_t se = beta == 1.0f ? cudaSuccess : launch_scale(sc);
        note_config(cfg);
        if (se != cudaSuccess) { note_launch_error(se); return GEMM_ERR_LAUNCH; }
        return GEMM_OK;
    }

    // k partition in multiples of the kernel's k slice (16); fewer splits than asked for when k is short
    const int64_t quantum = 16;
    const int64_t chunk = ((k + split_k - 1) / split_k + quantum - 1) / quantum * quantum;
    const int splits = (int)((k + chunk - 1) / chunk);

    // all partial sums must fit the fixed array
    const unsigned __int128 need = (unsigned __int128)splits * (unsigned __int128)m * (unsigned __int128)n * sizeof(float);
    if (need > (unsigned __int128)GEMM_STATIC_SCRATCH_BYTES) return GEMM_ERR_TOO_LARGE;

    float* scratch = nullptr;
    cudaError_t e = scratch_address(&scratch);
    if (e != cudaSuccess) { note_launch_error(e); return GEMM_ERR_LAUNCH; }

    GemmArgs a{GEMM_F32, ta, tb, m, n, k, alpha, beta, A, B, C, lda, ldb, ldc, static_cast<cudaStream_t>(stream), status};
    if (splits > 1) {
        // 64 x 64 CTA tiles: the problems that fit the array have few tiles, and the smallest tile spreads them
        // over the most SMs.  Every entry (split, i < m, j < n) of the scratch is written by this kernel before
        // the reduction reads it, so nothing has to be cleared between calls.
        e = launch_simt_fast(a, /*tile id of 64 x 64*/ 3, KSplit{splits, chunk}, scratch, &cfg);
        if (e == cudaSuccess) e = launch_splitk_reduce(a, splits, scratch);
        cfg.launches = 2;
    } else {
        // k no longer than one slice: a single pass with the epilogue fused, no scratch involved
        e = launch_simt_fast(a, 3, KSplit{1, chunk}, nullptr, &cfg);
        cfg.launches = 1;
    }
    note_config(cfg);
    if (e != cudaSuccess) { note_launch_error(e); return GEMM_ERR_LAUNCH; }
    return GEMM_OK;
}
