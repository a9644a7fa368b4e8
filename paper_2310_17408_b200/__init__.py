"""B200 (sm_100a) GEMM library: C <- alpha*op(A)*op(B) + beta*C, BLAS column-major.

The product is the CUDA shared library built from csrc/ (C ABI in include/b200_gemm.h); this
package is its thin Python binding.  Importing it without the built library raises ImportError.
"""
from .binding import *  # noqa: F401,F403
from .binding import (GemmConfig, EXPORTS, library_path, gemm, gemm_host, gemm_workspace_bytes,  # noqa: F401
                      gemm_set_workspace, gemm_last_config, gemm_force_kernel, gemm_force_tile,
                      gemm_poll_status, gemm_status_detail, gemm_status_string, gemm_last_cuda_error,
                      gemm_f32_splitk_static, GEMM_STATIC_SCRATCH_BYTES, gemm_selftest_wait_expiry,
                      ConvShape, conv_shape, conv2d_im2row, im2row, conv2d_workspace_bytes, conv2d_force_lowering)
