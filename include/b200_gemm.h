/*
 * b200_gemm.h — C ABI of the B200 (sm_100a) GEMM library.
 *
 * The library computes the operation the paper's BLIS-style algorithm computes (Section II-A:
 * C = C + A B through loops L1-L5, Pack-A / Pack-B and the mr x nr micro-kernel, Fig. 1), with
 * the alpha / beta scaling of the micro-kernel of Fig. 3 folded in:
 *
 *        C  <-  alpha * op(A) * op(B) + beta * C
 *
 * in BLAS column-major convention: element (i, j) of a stored matrix X is X[i + j*ldx].
 * Every matrix pointer is a DEVICE pointer unless a function says otherwise; scalars are passed
 * by value from the host.  No function throws, aborts or prints.
 */
#ifndef B200_GEMM_H
#define B200_GEMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* element types of A and B, and of C: fp32 unless the name says otherwise */
typedef enum {
    GEMM_F32  = 0,  /* A, B fp32; exact IEEE fp32 fused multiply-add arithmetic on the CUDA cores          */
    GEMM_F16  = 1,  /* A, B IEEE binary16; products accumulated in fp32 on the tensor cores (tcgen05/TMEM) */
    GEMM_BF16 = 2,  /* A, B bfloat16;      products accumulated in fp32 on the tensor cores                 */
    /* All-16-bit forms (Section III, "Data types": the generated f16 micro-kernel keeps A, B and C in 16-bit
     * storage).  A, B and C are of the one 16-bit type; products are still accumulated in fp32, and
     * alpha*acc + beta*C is rounded once, to nearest even, when it is stored.  Wherever this header says that C
     * is fp32, read "of the 16-bit type" for these two; ldc counts elements of that type. */
    GEMM_F16_C16  = 3,
    GEMM_BF16_C16 = 4,
    /* fp32 A, B and C multiplied on the tensor cores: every operand entry is split into three bfloat16 pieces
     * (x = x1 + x2 + x3 to within the last bit or two of x), and the six piece products that matter,
     * A1 B1 + A1 B2 + A2 B1 + A2 B2 + A1 B3 + A3 B1, are accumulated in fp32, smallest first.  Not the exact IEEE
     * fp32 arithmetic of GEMM_F32 (the dropped products are of relative size 2^-24; results stay within the same
     * error bound 4 k 2^-24 max|A| max|B| and are exact on small integers), but 1.4 to 3.4 times faster from about
     * 1280^3 on (where C has at least 16 tiles of 256 x 256 the six products run as one multiplication whose k loop
     * walks the pieces).  Needs a registered workspace of gemm_workspace_bytes(); without one, and for problems too small to
     * gain, the call runs as GEMM_F32.  Operands must be finite.  (The paper's data-type section, III-D, only
     * narrows the type; this mode goes the other way and keeps fp32 data on the narrow-type unit.) */
    GEMM_F32_TC   = 5,
    /* The paper's f16 arithmetic (Section III-D "Data types": with the precision set to f16 the generated micro-kernel
     * holds A, B, C and the accumulator registers in binary16).  A, B and C are binary16 and the products are
     * accumulated in binary16 on the tensor cores (tcgen05.mma with a binary16 accumulator); alpha*acc + beta*C is
     * formed in fp32 from the binary16 sum and rounded once, to nearest even, at the store.  The running sum is
     * rounded as the hardware rounds it, which need not be after every product as a scalar fp16 loop would: results
     * agree with such a loop to within 2 k 2^-11 sum_p |a_ip b_pj| and exactly while every partial sum is a
     * binary16 number.  Sums beyond 65504 overflow to infinity, as in any binary16 accumulation.  k is never split. */
    GEMM_F16_ACC16 = 6
} gemm_dtype_t;

/* return codes (0 = success; -1 .. -15 = the 1-based position of the first invalid argument of gemm()) */
enum {
    GEMM_OK            = 0,
    GEMM_ERR_WORKSPACE = -100,  /* a forced configuration needs more workspace than is registered      */
    GEMM_ERR_LAUNCH    = -101,  /* the CUDA runtime refused a launch; see gemm_last_cuda_error()        */
    GEMM_ERR_ARCH      = -102,  /* the current device is not compute capability 10.x                    */
    GEMM_ERR_DEVICE    = -103,  /* a bounded device-side wait expired (reported by gemm_poll_status())  */
    GEMM_ERR_TOO_LARGE = -104   /* a size exceeds what an entry point supports                          */
};

/* kernel families, as reported by gemm_last_config() and accepted by gemm_force_kernel() */
enum {
    GEMM_KERNEL_AUTO         = 0,
    GEMM_KERNEL_SIMT_GENERIC = 1,  /* any dtype, any alignment: bounds-checked scalar loads, fp32 FMA          */
    GEMM_KERNEL_SIMT_FAST    = 2,  /* fp32: register-blocked 8x8 FFMA micro-tiles, shared-memory double buffer */
    GEMM_KERNEL_TENSOR       = 3,  /* fp16/bf16: TMA -> swizzled shared memory -> tcgen05.mma -> TMEM          */
    GEMM_KERNEL_SIMT_DIRECT  = 4,  /* fp32, tiny problems: operands straight from global memory to registers   */
    GEMM_KERNEL_SCALE_ONLY   = 6   /* C <- beta*C (alpha == 0 or k == 0)                                        */
};

typedef struct {
    int32_t kernel;        /* one of GEMM_KERNEL_*                                           */
    int32_t tile_m;        /* CTA tile rows of C                                             */
    int32_t tile_n;        /* CTA tile columns of C                                          */
    int32_t tile_k;        /* k extent of one pipeline stage                                 */
    int32_t split_k;       /* number of k partitions (1 = none)                              */
    int32_t stages;        /* pipeline depth                                                 */
    int32_t grid;          /* CTAs launched for the main kernel                              */
    int32_t vector_a;      /* elements per global load of A (SIMT paths) / 1 if TMA operand  */
    int32_t vector_b;
    int32_t launches;      /* kernels enqueued by the call (main + reduction / scaling)      */
    int32_t repacked;      /* bit 0: A was copied to an aligned layout first, bit 1: B       */
    int32_t tail_split;    /* fp32: k ranges each tile of the last, partly filled wave was cut into (0 = not used) */
    int32_t lowering;      /* conv2d_im2row: one of CONV_LOWERING_* (0 for plain gemm calls)                        */
} gemm_config_t;

/*
 * gemm — the whole hot path: tile selection, the loops over n, m and k (Fig. 1, L1-L5), operand
 * staging into on-chip memory (the role of Pack-A / Pack-B), the rank-k update (micro-kernel, L6)
 * and the alpha / beta epilogue of Fig. 3 fused into the store of C.
 *
 *   dtype          gemm_dtype_t
 *   transA/transB  'N'/'n': op(X) = X;  'T'/'t'/'C'/'c': op(X) = X^T (real data)
 *   m, n, k        op(A) is m x k, op(B) is k x n, C is m x n; all >= 0
 *   A, lda         device pointer; stored m x k (lda >= max(1,m)) if transA = N, else k x m (lda >= max(1,k));
 *                  elements of `dtype`; never written
 *   B, ldb         device pointer; stored k x n (ldb >= max(1,k)) if transB = N, else n x k (ldb >= max(1,n))
 *   C, ldc         device pointer to fp32 (16-bit for the *_C16 types), m x n, ldc >= max(1,m); read only if beta != 0 (so NaN/Inf in C
 *                  do not propagate when beta == 0); rows m..ldc-1 of every column are never touched
 *   alpha, beta    fp32 scalars by value
 *   stream         cudaStream_t (NULL = the default stream)
 *
 * Any natural alignment of A, B, C and any legal leading dimension is accepted; 16-byte aligned pointers
 * with lda, ldb multiples of 16 bytes take the fast paths.  The call is asynchronous: work is enqueued on
 * `stream` and the buffers must stay valid until the stream has passed it.  C must not overlap A or B.
 * Quick returns: m == 0 or n == 0 does nothing; alpha == 0 or k == 0 computes C <- beta*C (beta == 0
 * stores +0 without reading C, beta == 1 does nothing), and A, B may then be NULL.
 * Returns GEMM_OK, or -(position of the first invalid argument) with nothing launched and C untouched,
 * or one of the GEMM_ERR_* codes.
 */
int gemm(int dtype, char transA, char transB, int64_t m, int64_t n, int64_t k,
         float alpha, const void* A, int64_t lda, const void* B, int64_t ldb,
         float beta, void* C, int64_t ldc, void* stream);

/*
 * gemm_strided_batched — `batch` independent problems of one shape in a single call:
 *        C_b  <-  alpha * op(A_b) * op(B_b) + beta * C_b,     b = 0 .. batch-1,
 * with X_b = X + b*strideX (strides in elements of the matrix's type; strideA and strideB may be 0 to share an
 * operand; strideC >= ldc*n so that results do not overlap).  Everything else as for gemm().
 * This is the small-problem end of the path.  The paper keeps a family of micro-kernels for problems its 8 x 12
 * kernel fits badly, among them a variant that skips packing altogether (Section III-B "Edge Cases": the
 * non-packed variant reads A where it lies, because for small problems the packing is not paid back); here
 * small fp32 problems (and every fp32 gemm() call below the same size) run in a kernel that reads its operands
 * from global memory straight into registers, without shared-memory staging, workspace or reduction pass, larger
 * ones share one launch of the register-blocked kernel.  16-bit batches whose operands TMA can address (16-byte
 * aligned A and B, lda, ldb, strideA and strideB multiples of 8 elements) run as ONE launch of the tensor-core
 * kernel, the problem index being the third coordinate of the operand maps; other small 16-bit problems share one
 * launch of the bounds-checked kernel, and what is left goes through gemm() one by one.
 * Returns GEMM_OK, -(position of the first invalid argument of THIS function; 10, 13, 17 = the strides, 18 = batch)
 * or a GEMM_ERR_* code.  Asynchronous on `stream`.
 */
int gemm_strided_batched(int dtype, char transA, char transB, int64_t m, int64_t n, int64_t k, float alpha,
                         const void* A, int64_t lda, int64_t strideA, const void* B, int64_t ldb, int64_t strideB,
                         float beta, void* C, int64_t ldc, int64_t strideC, int64_t batch, void* stream);

/*
 * gemm_host — the same operation on HOST buffers (pinned memory for full speed; pageable works but serialises).
 * Takes device buffers from a memory pool of the library's own (kept between calls; the application's default pool
 * is not touched), then moves column panels of op(B) and C through a three-stream pipeline (copy in / multiply on
 * `stream` / copy out), so that transfers overlap the arithmetic, and synchronises `stream` before returning.  While A
 * itself is still on its way the leading panels are multiplied k panel by k panel, each step adding onto C (the order of
 * the paper's loop L2, Fig. 1): a large result is therefore summed in a different order than gemm() sums it, inside
 * the same error bound (identical on integer-valued data).  Only the m x n window of C is transferred: C is copied
 * in only when beta != 0, and rows m..ldc-1 of the host array are never touched.  Leading dimensions and layout as for
 * gemm().  Calls from several host threads are serialised.
 */
int gemm_host(int dtype, char transA, char transB, int64_t m, int64_t n, int64_t k,
              float alpha, const void* A_host, int64_t lda, const void* B_host, int64_t ldb,
              float beta, void* C_host, int64_t ldc, void* stream);

/*
 * Workspace (device memory, caller-owned).  Split-k configurations keep fp32 partial sums there, and
 * operands whose leading dimension TMA cannot address are first copied there in an aligned layout
 * (the counterpart of the paper's packing buffers Ac / Bc).  Without a workspace, or with one that is
 * too small, gemm() silently picks a configuration that needs none.
 *   gemm_workspace_bytes  bytes the selector would like for this problem (0 = none)
 *   gemm_set_workspace    registers `dev` (>= 256-byte aligned) of `bytes` bytes on the current device for calls
 *                         made on `stream`; dev == NULL unregisters that entry.  A workspace registered with
 *                         stream == NULL serves every stream that has no workspace of its own.  The library never
 *                         frees or reallocates a workspace; it must stay valid while calls that may use it are
 *                         in flight.
 * Thread safety: gemm() may be called from several host threads at once.  Calls that share a workspace must be
 * ordered on one stream (the library does not order them); calls on distinct streams with distinct workspaces,
 * or that need none, are independent.
 */
size_t gemm_workspace_bytes(int dtype, char transA, char transB, int64_t m, int64_t n, int64_t k);
int gemm_set_workspace(void* dev, size_t bytes, void* stream);

/*
 * gemm_f32_splitk_static — fp32 split-k GEMM that allocates nothing.  (The paper has no counterpart: this is a
 * deployment variant of the split-k path of gemm(), not a step of its algorithm.)
 *
 * Who needs it: code that must not call cudaMalloc or any allocating routine around the GEMM.  Examples: a
 * plugin that runs inside another program's memory budget and is handed only its inputs and outputs; a control
 * or serving loop that cannot afford the device-wide synchronisation an allocation can cause; a thread from
 * which no allocator is reachable.  Such callers cannot give gemm() a workspace, and without one gemm() does
 * not split k, which leaves most SMs idle on problems with a small m*n and a large k.
 *
 * This entry point keeps the fp32 partial sums of the k partitions in a fixed array of GEMM_STATIC_SCRATCH_BYTES
 * that is part of the library image: every GPU that loads the library holds that much memory until the process
 * exits.  The caller passes only inputs and outputs (device pointers, fp32, layout and leading dimensions as
 * for gemm()); split_k in 2..64 is the number of k partitions asked for (fewer are used when k is short).
 *   - split_k * m * n * 4 bytes must fit the array; otherwise GEMM_ERR_TOO_LARGE is returned and nothing runs.
 *   - k >= 1; alpha and beta as for gemm(): C is not read when beta == 0, and alpha == 0 computes C <- beta*C
 *     without reading A or B (which may then be NULL).
 *   - The first call on each device looks up the array's device address (a symbol query, not an allocation).
 *     Make that first call outside any stream capture.
 *   - All calls share the one array, and it keeps what the previous call left in it.  Nothing has to be cleared:
 *     each call overwrites every partial sum that it later reads.  Two calls that may be on the GPU at the same
 *     time (different streams or host threads) race on the array: order them on one stream.
 * Returns GEMM_OK, -(position of the first invalid argument of THIS function: 1 = transA ... 14 = split_k;
 * gemm_status_string() names the positions of gemm() and does not apply), GEMM_ERR_TOO_LARGE, GEMM_ERR_ARCH or
 * GEMM_ERR_LAUNCH (then gemm_last_cuda_error() has the CUDA error).  gemm_last_config() reports the call.
 */
#define GEMM_STATIC_SCRATCH_BYTES (8u << 20)
int gemm_f32_splitk_static(char transA, char transB, int64_t m, int64_t n, int64_t k, float alpha,
                           const float* A, int64_t lda, const float* B, int64_t ldb, float beta, float* C, int64_t ldc,
                           int split_k, void* stream);

/*
 * Convolution layers lowered to GEMM with the im2row transform (Section IV-C, "Rectangular Matrices": the GEMM
 * dimensions of Tables "resnet50" and "vgg16" are m = batch*Ho*Wo output pixels, n = C_out, k = C_in*kh*kw).
 *
 *   conv2d_im2row   Y <- alpha * conv(X, W) + beta * Y, computed as the GEMM the lowering defines,
 *                       Y[C_out x pixels] = W[C_out x k] * L[k x pixels],
 *                   where column j = (b*Ho + ho)*Wo + wo of L is the receptive field of output pixel j:
 *                   L(p, j) = X(b, ho*stride_h - pad_h + r, wo*stride_w - pad_w + s, c) with p = (r*kw + s)*C_in + c,
 *                   and 0 where that position lies outside the image (zero padding).
 *                   Ho = (H + 2*pad_h - kh)/stride_h + 1, Wo likewise.
 *     X       device pointer, NHWC activations of `dtype`: element (b, h, w, c) at ((b*H + h)*W + w)*C_in + c
 *     W, ldw  device pointer, the filters as a column-major C_out x k matrix of `dtype` (ldw >= C_out), i.e.
 *             element (co; r, s, c) at co + ((r*kw + s)*C_in + c)*ldw
 *     Y, ldy  device pointer to fp32 (16-bit for the *_C16 types: a layer's result can then feed the next layer), NHWC result: element (co; pixel j) at co + j*ldy, ldy >= C_out; read only if
 *             beta != 0; rows C_out..ldy-1 are never touched
 *   Where it can, the lowering is fused into the operand staging of the GEMM kernels and L never exists in memory:
 *   fp32 reads X through the index map inside the SIMT kernel's loads; fp16/bf16 layers with C_in a multiple of
 *   64, a 16-byte aligned X, filters TMA can address (16-byte aligned W, ldw a multiple of 8), square filters and
 *   the same stride and padding in both directions let TMA's im2col mode deliver the swizzled tiles.  1 x 1 layers
 *   with stride 1 and no padding need no lowering (L is X).  All other fp16/bf16 layers first write L into the
 *   registered workspace with im2row() and then run gemm() on it; they return GEMM_ERR_WORKSPACE if the workspace
 *   is smaller than conv2d_workspace_bytes().  fp32 layers whose C_in is not a multiple of 4 (or whose X is not
 *   16-byte aligned) take that explicit route too when the workspace has room, because the index map then needs
 *   scalar loads; without room they stay fused.
 *   Returns GEMM_OK, -(position of the first invalid argument) (2 = a field of *shape), or a GEMM_ERR_* code.
 *   Asynchronous on `stream`, like gemm().
 *
 *   im2row          the transform by itself: writes L (element type of X, leading dimension ld >= k, column-major,
 *                   16-byte chunks when alignment allows) to `out`.  An HBM-bound copy: C_in*kh*kw*pixels elements.
 *                   Rows k..ld-1 of a column are either left untouched or set to zero.
 */
typedef struct {
    int64_t batch, h, w, c_in, c_out;
    int32_t kh, kw, stride_h, stride_w, pad_h, pad_w;
} conv_shape_t;

enum {
    CONV_LOWERING_NONE     = 0,
    CONV_LOWERING_FUSED    = 1,  /* index map / TMA im2col inside the GEMM kernel; L never materialised */
    CONV_LOWERING_EXPLICIT = 2,  /* im2row() into the workspace, then gemm()                             */
    CONV_LOWERING_IDENTITY = 3   /* 1 x 1, stride 1, no padding: L is X                                  */
};

int conv2d_im2row(int dtype, const conv_shape_t* shape, float alpha, const void* X, const void* W, int64_t ldw,
                  float beta, void* Y, int64_t ldy, void* stream);
int im2row(int dtype, const conv_shape_t* shape, const void* X, void* out, int64_t ld, void* stream);
/* workspace conv2d_im2row would like for this layer: the lowered matrix if it has to be written, plus what the GEMM asks for */
size_t conv2d_workspace_bytes(int dtype, const conv_shape_t* shape);
/* tests / benchmarks: 0 = choose, CONV_LOWERING_FUSED or CONV_LOWERING_EXPLICIT = take that route when it is possible */
int conv2d_force_lowering(int how);

/* configuration chosen by the most recent gemm() of the calling thread (for tests and reports) */
int gemm_last_config(gemm_config_t* out);

/* tests / benchmarks: force a kernel family (GEMM_KERNEL_AUTO restores the selector).  A forced family
 * that cannot run the problem (wrong dtype, alignment) falls back to the selector's choice.  The forcing
 * functions (these two and conv2d_force_lowering) act on the calling host thread only.
 * gemm_force_tile: force the tile (0 = auto) and split_k (0 = auto; 1 = no split of any kind) of the chosen family. */
int gemm_force_kernel(int kernel);
int gemm_force_tile(int tile_m, int tile_n, int split_k);
/* how a split of k is finished (fp32): 0 = choose; 1 = partial sums in the workspace and a separate reduction pass;
 * 2 = inside the main kernel: the CTAs that hold the k ranges of a tile run as one thread-block cluster and sum the
 * tile through distributed shared memory (at most 8 ranges, no workspace; a wish for more ranges is cut to 8) */
int gemm_force_reduction(int how);

/*
 * Device status.  Every wait inside the kernels (on an mbarrier) is bounded; a wait that expires
 * records a code in a device status word, the CTA drains and exits normally.  gemm_poll_status()
 * synchronises the device, returns GEMM_OK or GEMM_ERR_DEVICE and clears the word;
 * gemm_status_detail() returns the raw word of the last poll (role and barrier that gave up).
 */
int gemm_poll_status(void);
uint32_t gemm_status_detail(void);
/* Exercises the give-up path without a fault: enqueues a one-warp kernel that waits, with a limit of well under a
 * millisecond, on a barrier nothing arrives at.  The wait expires, the kernel exits normally, and the next
 * gemm_poll_status() returns GEMM_ERR_DEVICE with detail 0xE57F01xx; the context stays usable. */
int gemm_selftest_wait_expiry(void* stream);
const char* gemm_status_string(int code);
int gemm_last_cuda_error(void);   /* cudaError_t of the last failed launch, 0 if none */

/*
 * Peak-confirmation probes.  The paper measures its micro-kernels in "solo mode" (Section IV-A: the micro-kernel
 * called repeatedly on operands that stay in the fastest memory, apart from the GEMM around it).  These are the
 * counterparts for the three units that bound the kernels of this library; a benchmark calls them on the device
 * it reports on and quotes the results beside the peaks it divides by.  Each call runs its kernel twice on
 * `stream` (once to warm up, once between two CUDA events), synchronises, and returns the rate of the timed run.
 * Run times are bounded by the caps on the iteration counts (at most a few hundred milliseconds).
 *
 *   gemm_probe_copy   streams `bytes` (a multiple of 16, at most 64 GiB) from src to dst (device pointers, 16-byte
 *                     aligned, not overlapping; dst is overwritten).  *gbs = (bytes read + bytes written) / time, GB/s.
 *   gemm_probe_ffma   fp32 fused multiply-adds on all SMs, no global memory traffic.  pattern 0: 16 independent
 *                     register-only chains per thread, 2048 threads per SM (the issue-rate ceiling); pattern 1: the
 *                     micro-kernel of the SIMT GEMM kernel on its own, an 8 x 8 block of accumulators per thread updated
 *                     by outer products whose operands are read from shared memory with the kernel's 128-bit fragment
 *                     loads, 2 x 256 threads per SM, scalar FMAs; pattern 2: the same on packed fma.rn.f32x2 in the
 *                     kernel's arrangement.  iters in 1..65536 loop trips of 8 steps each.  *tflops = 2 * FMAs / time.
 *   gemm_probe_umma   tcgen05.mma (kind::f16, fp32 accumulators in TMEM) on operand tiles that stay in shared memory:
 *                     one CTA per SM issuing 128 x 256 x 16 MMAs (pair = 0), or one CTA pair per two SMs issuing
 *                     256 x 256 x 16 MMAs with cta_group::2 (pair = 1); dtype GEMM_F16 or GEMM_BF16; kblocks in
 *                     1..262144 blocks of four MMAs (k = 64).  *tflops = 2*M*N*K per MMA / time.  Its waits are
 *                     bounded like all others; an expiry shows in gemm_poll_status().
 *   ms (may be NULL) receives the duration of the timed run in milliseconds.
 * Return GEMM_OK, -(position of the first invalid argument), GEMM_ERR_ARCH or GEMM_ERR_LAUNCH.
 */
int gemm_probe_copy(void* dst, const void* src, size_t bytes, double* gbs, double* ms, void* stream);
int gemm_probe_ffma(int pattern, int iters, double* tflops, double* ms, void* stream);
int gemm_probe_umma(int dtype, int pair, int kblocks, double* tflops, double* ms, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* B200_GEMM_H */
