"""ctypes binding of libb200gemm.so: the same names and argument order as include/b200_gemm.h.

Argument marshalling only.  Pointers are plain integers (torch `tensor.data_ptr()`, numpy
`array.ctypes.data`); `stream` is a cudaStream_t as an integer (`torch.cuda.current_stream().cuda_stream`).
There is no fallback: importing this module without the built CUDA library raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

_LIB_PATH = Path(__file__).resolve().parent / "libb200gemm.so"

GEMM_F32, GEMM_F16, GEMM_BF16, GEMM_F16_C16, GEMM_BF16_C16, GEMM_F32_TC, GEMM_F16_ACC16 = 0, 1, 2, 3, 4, 5, 6
GEMM_OK = 0
GEMM_ERR_WORKSPACE, GEMM_ERR_LAUNCH, GEMM_ERR_ARCH, GEMM_ERR_DEVICE, GEMM_ERR_TOO_LARGE = -100, -101, -102, -103, -104
GEMM_KERNEL_AUTO, GEMM_KERNEL_SIMT_GENERIC, GEMM_KERNEL_SIMT_FAST, GEMM_KERNEL_TENSOR = 0, 1, 2, 3
GEMM_KERNEL_SIMT_DIRECT = 4
GEMM_KERNEL_SCALE_ONLY = 6

EXPORTS = ("gemm", "gemm_host", "gemm_workspace_bytes", "gemm_set_workspace", "gemm_last_config",
           "gemm_force_kernel", "gemm_force_tile", "gemm_poll_status", "gemm_status_detail",
           "gemm_status_string", "gemm_last_cuda_error", "gemm_f32_splitk_static",
           "gemm_selftest_wait_expiry", "conv2d_im2row", "im2row", "conv2d_workspace_bytes",
           "conv2d_force_lowering", "gemm_strided_batched", "gemm_force_reduction", "gemm_probe_copy", "gemm_probe_ffma", "gemm_probe_umma")
CONV_LOWERING_NONE, CONV_LOWERING_FUSED, CONV_LOWERING_EXPLICIT, CONV_LOWERING_IDENTITY = 0, 1, 2, 3
GEMM_STATIC_SCRATCH_BYTES = 8 << 20


class GemmConfig(ctypes.Structure):
    _fields_ = [(name, ctypes.c_int32) for name in
                ("kernel", "tile_m", "tile_n", "tile_k", "split_k", "stages", "grid", "vector_a", "vector_b",
                 "launches", "repacked", "tail_split", "lowering")]

    def as_dict(self):
        return {name: getattr(self, name) for name, _ in self._fields_}


class ConvShape(ctypes.Structure):
    """conv_shape_t of the header: NHWC activations batch x h x w x c_in, c_out filters of kh x kw, strides, zero padding."""
    _fields_ = [("batch", ctypes.c_int64), ("h", ctypes.c_int64), ("w", ctypes.c_int64), ("c_in", ctypes.c_int64),
                ("c_out", ctypes.c_int64), ("kh", ctypes.c_int32), ("kw", ctypes.c_int32),
                ("stride_h", ctypes.c_int32), ("stride_w", ctypes.c_int32), ("pad_h", ctypes.c_int32),
                ("pad_w", ctypes.c_int32)]


def _load() -> ctypes.CDLL:
    if not _LIB_PATH.exists():
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python paper_2310_17408_b200/build.py` "
                          "(nvcc, sm_100a); this package has no CPU or library fallback")
    lib = ctypes.CDLL(str(_LIB_PATH), mode=ctypes.RTLD_LOCAL)
    i64, vp, ci, cf, cc = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_char
    sig = [ci, cc, cc, i64, i64, i64, cf, vp, i64, vp, i64, cf, vp, i64, vp]
    lib.gemm.restype = ci
    lib.gemm.argtypes = sig
    lib.gemm_host.restype = ci
    lib.gemm_host.argtypes = sig
    lib.gemm_workspace_bytes.restype = ctypes.c_size_t
    lib.gemm_workspace_bytes.argtypes = [ci, cc, cc, i64, i64, i64]
    lib.gemm_set_workspace.restype = ci
    lib.gemm_set_workspace.argtypes = [vp, ctypes.c_size_t, vp]
    lib.gemm_last_config.restype = ci
    lib.gemm_last_config.argtypes = [ctypes.POINTER(GemmConfig)]
    lib.gemm_force_kernel.restype = ci
    lib.gemm_force_kernel.argtypes = [ci]
    lib.gemm_force_tile.restype = ci
    lib.gemm_force_tile.argtypes = [ci, ci, ci]
    lib.gemm_poll_status.restype = ci
    lib.gemm_poll_status.argtypes = []
    lib.gemm_status_detail.restype = ctypes.c_uint32
    lib.gemm_status_detail.argtypes = []
    lib.gemm_status_string.restype = ctypes.c_char_p
    lib.gemm_status_string.argtypes = [ci]
    lib.gemm_last_cuda_error.restype = ci
    lib.gemm_last_cuda_error.argtypes = []
    lib.gemm_selftest_wait_expiry.restype = ci
    lib.gemm_selftest_wait_expiry.argtypes = [vp]
    sp = ctypes.POINTER(ConvShape)
    lib.conv2d_im2row.restype = ci
    lib.conv2d_im2row.argtypes = [ci, sp, cf, vp, vp, i64, cf, vp, i64, vp]
    lib.im2row.restype = ci
    lib.im2row.argtypes = [ci, sp, vp, vp, i64, vp]
    lib.conv2d_workspace_bytes.restype = ctypes.c_size_t
    lib.conv2d_workspace_bytes.argtypes = [ci, sp]
    lib.conv2d_force_lowering.restype = ci
    lib.conv2d_force_lowering.argtypes = [ci]
    lib.gemm_f32_splitk_static.restype = ci
    lib.gemm_f32_splitk_static.argtypes = [cc, cc, i64, i64, i64, cf, vp, i64, vp, i64, cf, vp, i64, ci, vp]
    lib.gemm_strided_batched.restype = ci
    lib.gemm_strided_batched.argtypes = [ci, cc, cc, i64, i64, i64, cf, vp, i64, i64, vp, i64, i64, cf, vp, i64, i64, i64, vp]
    lib.gemm_force_reduction.restype = ci
    lib.gemm_force_reduction.argtypes = [ci]
    dp = ctypes.POINTER(ctypes.c_double)
    lib.gemm_probe_copy.restype = ci
    lib.gemm_probe_copy.argtypes = [vp, vp, ctypes.c_size_t, dp, dp, vp]
    lib.gemm_probe_ffma.restype = ci
    lib.gemm_probe_ffma.argtypes = [ci, ci, dp, dp, vp]
    lib.gemm_probe_umma.restype = ci
    lib.gemm_probe_umma.argtypes = [ci, ci, ci, dp, dp, vp]
    return lib


_lib = _load()


def library_path() -> str:
    return str(_LIB_PATH)


def _c(flag) -> bytes:
    b = flag.encode() if isinstance(flag, str) else bytes(flag)
    if len(b) != 1:
        raise ValueError("trans flag must be one character")
    return b


def gemm(dtype, transA, transB, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, stream=0) -> int:
    return _lib.gemm(dtype, _c(transA), _c(transB), m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, stream)


def gemm_host(dtype, transA, transB, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, stream=0) -> int:
    return _lib.gemm_host(dtype, _c(transA), _c(transB), m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, stream)


def gemm_strided_batched(dtype, transA, transB, m, n, k, alpha, A, lda, strideA, B, ldb, strideB, beta, C, ldc, strideC,
                         batch, stream=0) -> int:
    return _lib.gemm_strided_batched(dtype, _c(transA), _c(transB), m, n, k, alpha, A, lda, strideA, B, ldb, strideB,
                                     beta, C, ldc, strideC, batch, stream)


def gemm_force_reduction(how) -> int:
    return _lib.gemm_force_reduction(how)


def gemm_workspace_bytes(dtype, transA, transB, m, n, k) -> int:
    return int(_lib.gemm_workspace_bytes(dtype, _c(transA), _c(transB), m, n, k))


def gemm_set_workspace(dev_ptr, nbytes, stream=0) -> int:
    return _lib.gemm_set_workspace(dev_ptr, nbytes, stream)


def gemm_last_config() -> dict:
    cfg = GemmConfig()
    _lib.gemm_last_config(ctypes.byref(cfg))
    return cfg.as_dict()


def gemm_force_kernel(kernel) -> int:
    return _lib.gemm_force_kernel(kernel)


def gemm_force_tile(tile_m, tile_n, split_k) -> int:
    return _lib.gemm_force_tile(tile_m, tile_n, split_k)


def gemm_poll_status() -> int:
    return _lib.gemm_poll_status()


def gemm_status_detail() -> int:
    return int(_lib.gemm_status_detail())


def gemm_status_string(code) -> str:
    return _lib.gemm_status_string(code).decode()


def gemm_last_cuda_error() -> int:
    return _lib.gemm_last_cuda_error()


def gemm_f32_splitk_static(transA, transB, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, split_k, stream=0) -> int:
    """fp32 split-k GEMM whose partial sums live in a fixed array inside the library: it allocates nothing.
    Meant for callers that cannot allocate device memory or register a workspace (see include/b200_gemm.h)."""
    return _lib.gemm_f32_splitk_static(_c(transA), _c(transB), m, n, k, alpha, A, lda, B, ldb, beta, C, ldc,
                                       split_k, stream)


def gemm_selftest_wait_expiry(stream=0) -> int:
    """Enqueue the kernel whose bounded wait is certain to expire; gemm_poll_status() then reports GEMM_ERR_DEVICE."""
    return _lib.gemm_selftest_wait_expiry(stream)


def conv_shape(batch, h, w, c_in, c_out, kh, kw, stride_h=1, stride_w=1, pad_h=0, pad_w=0) -> ConvShape:
    return ConvShape(batch, h, w, c_in, c_out, kh, kw, stride_h, stride_w, pad_h, pad_w)


def conv2d_im2row(dtype, shape: ConvShape, alpha, X, W, ldw, beta, Y, ldy, stream=0) -> int:
    return _lib.conv2d_im2row(dtype, ctypes.byref(shape), alpha, X, W, ldw, beta, Y, ldy, stream)


def im2row(dtype, shape: ConvShape, X, out, ld, stream=0) -> int:
    return _lib.im2row(dtype, ctypes.byref(shape), X, out, ld, stream)


def conv2d_workspace_bytes(dtype, shape: ConvShape) -> int:
    return int(_lib.conv2d_workspace_bytes(dtype, ctypes.byref(shape)))


def conv2d_force_lowering(how) -> int:
    return _lib.conv2d_force_lowering(how)


def _probe(fn, *args):
    rate, ms = ctypes.c_double(0.0), ctypes.c_double(0.0)
    rc = fn(*args[:-1], ctypes.byref(rate), ctypes.byref(ms), args[-1])
    return rc, rate.value, ms.value


def gemm_probe_copy(dst, src, nbytes, stream=0):
    """(rc, GB/s, ms) of the library's streaming copy between two device buffers."""
    return _probe(_lib.gemm_probe_copy, dst, src, nbytes, stream)


def gemm_probe_ffma(pattern, iters, stream=0):
    """(rc, TFLOP/s, ms) of the fp32 FMA probes (pattern 0: register-only chains; 1 / 2: the SIMT kernel's 8 x 8 micro-kernel
    fed from shared memory, scalar / packed)."""
    return _probe(_lib.gemm_probe_ffma, pattern, iters, stream)


def gemm_probe_umma(dtype, pair, kblocks, stream=0):
    """(rc, TFLOP/s, ms) of tcgen05.mma on shared-memory-resident operands (pair = 1: CTA pairs, 256-row MMAs)."""
    return _probe(_lib.gemm_probe_umma, dtype, pair, kblocks, stream)
