"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import paper_2310_17408_b200 as g

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "b200_gemm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"^\s*(?:const\s+char\s*\*|int|size_t|uint32_t)\s+((?:gemm|conv2d|im2row)\w*)\s*\(", text, flags=re.M)
    return sorted(set(names))


def test_every_declared_symbol_is_exported():
    lib = ctypes.CDLL(g.library_path())
    names = declared_functions()
    assert "gemm" in names and "gemm_host" in names and len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(g.EXPORTS) == names


def test_argument_checks_run_without_a_device():
    # validation happens before any CUDA call: negative position of the first bad argument
    assert g.gemm(7, "N", "N", 1, 1, 1, 1.0, 16, 1, 16, 1, 0.0, 16, 1) == -1
    assert g.gemm(0, "N", "N", 4, 4, 4, 1.0, 16, 3, 16, 4, 0.0, 16, 4) == -9
    assert g.gemm(0, "N", "N", 4, 4, 4, 1.0, 16, 4, 16, 4, 0.0, 16, 2) == -14
    assert g.gemm(0, "N", "N", 0, 4, 4, 1.0, 0, 1, 0, 4, 0.0, 0, 1) == 0       # m == 0: nothing to do
    # the all-16-bit types are accepted by the same checks; 5 is not a type; C must be aligned to its own element size
    assert g.gemm(g.GEMM_F16_C16, "N", "N", 4, 4, 4, 1.0, 16, 4, 16, 4, 0.0, 16, 2) == -14
    assert g.gemm(g.GEMM_BF16_C16, "N", "N", 4, 4, 4, 1.0, 16, 4, 16, 4, 0.0, 17, 4) == -13
    assert g.gemm(g.GEMM_BF16, "N", "N", 4, 4, 4, 1.0, 16, 4, 16, 4, 0.0, 18, 4) == -13       # fp32 C at a 2-byte boundary
    assert g.gemm(9, "N", "N", 4, 4, 4, 1.0, 16, 4, 16, 4, 0.0, 16, 4) == -1
    assert "lda" in g.gemm_status_string(-9)
    assert g.gemm_force_kernel(99) == -1 and g.gemm_force_kernel(0) == 0


def test_convolution_argument_checks_run_without_a_device():
    s = g.conv_shape(1, 4, 4, 4, 4, 5, 5, 1, 1, 0, 0)              # filter larger than the padded image
    assert g.conv2d_im2row(0, s, 1.0, 16, 16, 4, 0.0, 16, 4) == -2
    s = g.conv_shape(2, 8, 8, 4, 6, 3, 3, 1, 1, 1, 1)
    assert g.conv2d_im2row(9, s, 1.0, 16, 16, 6, 0.0, 16, 6) == -1
    assert g.conv2d_im2row(0, s, 1.0, 16, 16, 5, 0.0, 16, 6) == -6
    assert g.im2row(0, s, 16, 16, 35) == -5                         # ld < k = 36
    assert g.conv2d_force_lowering(7) == -1 and g.conv2d_force_lowering(0) == 0
    # nothing to compute: an empty batch or no output channels succeed without touching anything
    assert g.conv2d_im2row(0, g.conv_shape(0, 8, 8, 4, 6, 3, 3, 1, 1, 1, 1), 1.0, 0, 16, 6, 0.0, 0, 6) == 0
    assert g.conv2d_im2row(2, g.conv_shape(2, 8, 8, 4, 0, 3, 3, 1, 1, 1, 1), 1.0, 16, 0, 1, 0.0, 0, 1) == 0
    assert g.im2row(0, g.conv_shape(0, 8, 8, 4, 6, 3, 3, 1, 1, 1, 1), 0, 0, 36) == 0
    # a layer whose lowered matrix must be written asks for room for it: k = 27 padded to 32 rows, 2 bytes each
    s = g.conv_shape(4, 32, 32, 3, 64, 3, 3, 1, 1, 1, 1)
    assert g.conv2d_workspace_bytes(2, s) >= 32 * 4 * 32 * 32 * 2
    assert g.conv2d_workspace_bytes(0, s) >= 32 * 4 * 32 * 32 * 4         # fp32 with 3 channels: lowered first, too
    s = g.conv_shape(4, 32, 32, 8, 64, 3, 3, 1, 1, 1, 1)
    assert g.conv2d_workspace_bytes(0, s) == g.gemm_workspace_bytes(0, "N", "N", 64, 4 * 32 * 32, 72)   # fp32, C_in % 4 == 0: fused


def test_workspace_request_for_split_k_shapes():
    # large-k, few-tile fp32 problem: the selector wants room for fp32 partial sums
    assert g.gemm_workspace_bytes(0, "N", "N", 256, 256, 65536) >= 2 * 256 * 256 * 4
    assert g.gemm_workspace_bytes(0, "N", "N", 8192, 8192, 8192) == 0
    assert g.gemm_workspace_bytes(0, "N", "N", 0, 8, 8) == 0
