// Internal interfaces between the translation units of the GEMM library (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "../../include/b200_gemm.h"

namespace b200gemm {

// Index map of the im2row lowering (Section IV-C): when a call carries one, op(B) is not read from memory as a
// stored matrix; its element (p, j) is the activation X(b, ho*sh - ph + r, wo*sw - pw + s, c) of an NHWC tensor, with
// j = (b*Ho + ho)*Wo + wo and p = (r*kw + s)*C_in + c, and zero where the receptive field leaves the image.
struct ConvIndex {
    const void* X;             // NHWC activations, element type of the call
    int64_t h, w, c_in;
    int32_t ho, wo, kh, kw, sh, sw, ph, pw;
};

struct GemmArgs {
    int dtype;
    bool ta, tb;           // op(X) = X^T ?
    int64_t m, n, k;
    float alpha, beta;
    const void* A;
    const void* B;
    float* C;
    int64_t lda, ldb, ldc;
    cudaStream_t stream;
    uint32_t* status;      // device status word (bounded waits report here)
    const ConvIndex* conv = nullptr;   // non-null: op(B) is the lowered activation matrix of this layer (B, ldb, tb unused)
    int out16 = 0;                     // element type of C: 0 = fp32, GEMM_F16 / GEMM_BF16 = that 16-bit type (C then points to it)
    int acc16 = 0;                     // binary16 inputs, binary16 accumulation on the tensor cores, binary16 result (GEMM_F16_ACC16)
    int ct = 0;                        // tensor kernels: the roles of the operands were exchanged; C (m x n here) is stored as its
                                       // transpose: element (i, j) at C[j + i*ldc]
    int split3 = 0;                    // fp32 operands: multiply on the tensor cores as three bfloat16 pieces each (GEMM_F32_TC)
    int64_t seg_k = 0;                 // CTA-pair kernel: A and B hold three bfloat16 pieces each, one after the other along k
                                       // (seg_k entries of k per piece, a multiple of 64, zero padded; k = 3 * seg_k)
};

// The all-16-bit data types (GEMM_F16_C16, GEMM_BF16_C16) are a 16-bit input type plus a 16-bit result:
// inside the library dtype is always the input type and out16 names the result's type.
inline int input_dtype(int dtype) {
    return (dtype == GEMM_F16_C16 || dtype == GEMM_F16_ACC16) ? GEMM_F16
           : (dtype == GEMM_BF16_C16 ? GEMM_BF16 : (dtype == GEMM_F32_TC ? GEMM_F32 : dtype));
}
inline int output16(int dtype) {
    return (dtype == GEMM_F16_C16 || dtype == GEMM_F16_ACC16) ? GEMM_F16 : (dtype == GEMM_BF16_C16 ? GEMM_BF16 : 0);
}
inline int c_elem_size(int dtype) { return output16(dtype) ? 2 : 4; }

// fp32 <-> the 16-bit result types, round to nearest even (device)
#ifdef __CUDACC__
__device__ __forceinline__ uint16_t f32_to_bits16(float v, int out16) {
    return out16 == GEMM_F16 ? __half_as_ushort(__float2half_rn(v)) : __bfloat16_as_ushort(__float2bfloat16_rn(v));
}
__device__ __forceinline__ float bits16_to_f32(uint16_t b, int out16) {
    return out16 == GEMM_F16 ? __half2float(__ushort_as_half(b)) : __bfloat162float(__ushort_as_bfloat16(b));
}
// element i of C in either representation
__device__ __forceinline__ float load_c(const float* C, int out16, int64_t i) {
    return out16 ? bits16_to_f32(reinterpret_cast<const uint16_t*>(C)[i], out16) : C[i];
}
__device__ __forceinline__ void store_c(float* C, int out16, int64_t i, float v) {
    if (out16) reinterpret_cast<uint16_t*>(C)[i] = f32_to_bits16(v, out16);
    else C[i] = v;
}
#endif

// k partition used by every split-k path: split s covers [s*chunk, min(k, (s+1)*chunk))
struct KSplit {
    int splits;
    int64_t chunk;
};

// device status word layout: bits 31..24 = 0xE5 marker, 23..16 = role, 15..8 = barrier id, 7..0 = stage
constexpr uint32_t STATUS_MARK = 0xE5000000u;

// Tail split of the fp32 SIMT path: tiles first .. are cut into `splits` k ranges of `chunk` each
// (first = INT_MAX: off).  Item i >= first writes its raw block to partials + (i - first) * tile_m * tile_n.
struct TailSplit {
    int first;
    int splits;
    int64_t chunk;
    float* partials;
};

// Extras of the fp32 SIMT kernel beyond one plain GEMM.
//   cluster_reduce  split-k finished inside the kernel: the CTAs that hold the k ranges of one tile are launched as one
//                   thread-block cluster (gridDim.z = cluster size <= 8).  Each leaves its partial sums in its own
//                   shared memory; after a cluster barrier every CTA sums one slice of the tile over all CTAs, in
//                   increasing split index, through distributed shared memory, applies alpha / beta and writes C.
//                   No workspace, no second launch; the hardware co-schedules a cluster, so the barrier cannot hang.
//   stride*         strided batch (batched kernel only): blockIdx.y is the problem index
struct SimtExtra {
    TailSplit tail;
    int cluster_reduce;
    int64_t strideA, strideB, strideC;
};
constexpr int CLUSTER_REDUCE_MAX_SPLITS = 8;      // portable cluster size

// Tile order shared by the kernels: groups of `group` tile rows, all tile columns inside a group, rows fastest,
// so that the CTAs resident at one time share their A and B panels in L2.
constexpr int SIMT_GROUP = 16;
__host__ __device__ inline void decode_tile(int tile, int tiles_m, int tiles_n, int* tm, int* tn, int group = SIMT_GROUP) {
    const int per_group = group * tiles_n;
    const int g = tile / per_group;
    const int rest = tiles_m - g * group;
    const int gsz = rest < group ? rest : group;
    *tm = g * group + (tile % per_group) % gsz;
    *tn = (tile % per_group) / gsz;
}

inline int elem_size(int dtype) { return (dtype == GEMM_F32 || dtype == GEMM_F32_TC) ? 4 : 2; }      // of A and B

// C <- beta*C  (beta == 0: store +0 without reading)
cudaError_t launch_scale(const GemmArgs& a, int64_t strideC = 0, int64_t batch = 1);

// generic bounds-checked SIMT kernel, any dtype / trans / alignment
cudaError_t launch_simt_generic(const GemmArgs& a, gemm_config_t* cfg, int64_t strideA = 0, int64_t strideB = 0,
                                int64_t strideC = 0, int64_t batch = 1);

// fp32 without operand staging (tiny problems; a strided batch of them): every thread reads its operands from global memory
cudaError_t launch_simt_direct(const GemmArgs& a, int64_t strideA, int64_t strideB, int64_t strideC, int64_t batch,
                               gemm_config_t* cfg);

// fast fp32 SIMT kernel.  tile: 0 = 128x128, 1 = 128x64, 2 = 64x128, 3 = 64x64.
// ks.splits > 1: raw partial sums go to `partials` ([split][n][m], fp32), no epilogue.
bool simt_fast_eligible(const GemmArgs& a, int* va, int* vb);
bool simt_fast_can_cluster_reduce(int tile);      // can this CTA tile finish a split of k inside the kernel?
cudaError_t launch_simt_fast(const GemmArgs& a, int tile, KSplit ks, float* partials, gemm_config_t* cfg,
                             TailSplit tail = TailSplit{0x7FFFFFFF, 1, 0, nullptr}, bool cluster_reduce = false);
// batch problems of identical shape, operands strideA / strideB / strideC elements apart (no split of k)
cudaError_t launch_simt_fast_batched(const GemmArgs& a, int tile, int64_t strideA, int64_t strideB, int64_t strideC,
                                     int64_t batch, gemm_config_t* cfg);
// finishes the tail tiles (bm x bn, tile order with groups of `group` rows):
// C <- alpha * sum_z slot[(t - first) * splits + z] + beta*C for tiles t >= first
cudaError_t launch_tail_reduce(const GemmArgs& a, int bm, int bn, int group, TailSplit tail);

// C <- alpha * sum_s partials[s] + beta*C, summed in increasing s (deterministic)
cudaError_t launch_splitk_reduce(const GemmArgs& a, int splits, const float* partials);

// tcgen05 tensor-core kernel (fp16 / bf16).  tile_n in {64, 128, 256}; tile_m is 128.
bool tensor_eligible(const GemmArgs& a);
// cluster: the ks.splits (2 .. 8) k ranges of a tile run as one thread-block cluster and sum the tile themselves through
// distributed shared memory (no partials, no reduction pass)
cudaError_t launch_tensor(const GemmArgs& a, int tile_n, KSplit ks, float* partials, gemm_config_t* cfg, bool cluster = false);
// the same on CTA pairs (tcgen05 cta_group::2): 256 x 256 tiles, two SMs per tile
cudaError_t launch_tensor_batched(const GemmArgs& a, int tile_n, int64_t strideA, int64_t strideB, int64_t strideC,
                                  int64_t batch, gemm_config_t* cfg);
cudaError_t launch_tensor_pair(const GemmArgs& a, KSplit ks, float* partials, gemm_config_t* cfg);

// copy op-independent stored matrix (rows x cols, ld) of 16-bit elements into an aligned layout (ld_out)
cudaError_t launch_repack16(const void* src, int64_t rows, int64_t cols, int64_t ld, void* dst, int64_t ld_out,
                            cudaStream_t stream);

// fp32 stored matrix (rows x cols, ld) -> three bfloat16 matrices p1, p2, p3 (leading dimension ld_p) with
// x = p1 + p2 + p3 up to the last bit or two of x: p1 = bf16(x), p2 = bf16(x - p1), p3 = bf16(x - p1 - p2)
cudaError_t launch_split3(const float* src, int64_t rows, int64_t cols, int64_t ld, void* p1, void* p2, void* p3,
                          int64_t ld_p, cudaStream_t stream, int64_t rows_out = 0, int64_t cols_out = 0);

// launches a one-warp kernel whose bounded wait is certain to expire (nothing arrives at its barrier)
cudaError_t launch_wait_expiry_probe(uint32_t* status, cudaStream_t stream);

int sm_count();
// status word of the current device and whether it is compute capability 10.x; false if the device cannot be queried
bool device_info(uint32_t** status, bool* arch_ok);

// runs one GEMM (possibly with an im2row index map in a.conv) through the selector on the current device;
// the first ws_skip bytes of the registered workspace are left alone
int dispatch_gemm(const GemmArgs& a, size_t ws_skip);
bool registered_workspace(cudaStream_t stream, void** ws, size_t* bytes);   // the one a call on `stream` may use
void note_lowering(int how);             // recorded in the calling thread's last configuration
void note_launch_error(cudaError_t e);
void note_config(const gemm_config_t& cfg);   // becomes the calling thread's gemm_last_config()
// whether TMA's im2col mode can do the lowering of this layer (defined with the tensor kernels)
bool conv_tma_eligible(int dtype, const ConvIndex& cv, int64_t batch);

}  // namespace b200gemm
