"""Parity of the convolution front end (conv2d_im2row, im2row; through the C ABI) with the CPU oracle's definition
of the layer.  Every route is covered: the lowering fused into the fp32 SIMT kernel's loads, TMA im2col mode on
the tensor path (single-CTA and CTA-pair kernels), the explicit im2row pass followed by gemm, and 1 x 1 layers
that need no lowering.  Tolerances are those of the GEMM it lowers to (k = kh*kw*C_in): bit-exact on
integer-valued inputs, fp32 max error <= 4*2^-24*(k*|alpha|*max|X|*max|W| + |beta|*max|Y0|), fp16/bf16 relative
Frobenius error <= 1e-3 against the fp64 oracle on the same rounded inputs."""
import numpy as np
import pytest
import torch

import oracle
import paper_2310_17408_b200 as g
from workloads import DTYPE_BF16, DTYPE_F16, DTYPE_F32, ConvProblem, conv_layer_problems

from gpu_util import drop_workspace, ensure_workspace, to_device

pytestmark = pytest.mark.gpu

# batch, h, w, c_in, c_out, kh, kw, stride, pad
SMALL = [
    (2, 7, 9, 3, 5, 3, 3, 1, 1),          # C_in = 3: scalar index map (fp32) / explicit lowering (16-bit)
    (1, 12, 10, 4, 6, 7, 7, 2, 3),
    (3, 5, 5, 8, 4, 1, 1, 1, 0),          # 1 x 1: identity lowering
    (2, 9, 8, 12, 70, 3, 3, 2, 0),
    (2, 13, 11, 64, 96, 3, 3, 1, 1),      # C_in % 64 == 0: TMA im2col; 286 pixels: tiles span rows and images
    (3, 10, 10, 128, 136, 3, 3, 2, 1),
    (1, 20, 17, 64, 40, 5, 5, 1, 2),
    (2, 6, 6, 192, 260, 1, 1, 2, 0),      # 1 x 1 with stride 2: a real gather
    (2, 24, 25, 64, 48, 3, 3, 1, 1),      # 1200 pixels, 48 output channels (half-empty MMA rows on the tensor path)
    (1, 70, 66, 128, 64, 3, 3, 2, 1),     # exactly 64 output channels, stride 2, 1155 pixels (ragged last tile)
    (1, 5, 150, 3, 4, 3, 3, 2, 1),        # a long image row with few channels
    (2, 4, 70, 5, 3, 5, 5, 1, 2),         # 70 per row, C_in = 5, wide filter
]


@pytest.fixture(autouse=True)
def _reset():
    yield
    g.conv2d_force_lowering(0)
    g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
    g.gemm_force_tile(0, 0, 0)


def geom_of(p):
    return oracle.conv_geom(p.batch, p.h, p.w, p.c_in, p.c_out, p.kh, p.kw, p.stride, p.stride, p.pad, p.pad)


def shape_of(p):
    return g.conv_shape(p.batch, p.h, p.w, p.c_in, p.c_out, p.kh, p.kw, p.stride, p.stride, p.pad, p.pad)


def make(gm, dtype, kind=None, alpha=1.0, beta=0.0, seed=5, ld_pad=(0, 0)):
    b, h, w, ci, co, kh, kw, st, pd = gm
    kinds = dict(kindX=kind, kindW=kind, kindY=kind) if kind else {}
    return ConvProblem("t", dtype, b, h, w, ci, co, kh, kw, st, pd, alpha, beta, seed=seed, ld_pad=ld_pad, **kinds)


def run_conv(p, X, W, Y0):
    ensure_workspace(g.conv2d_workspace_bytes(p.dtype, shape_of(p)) + (64 << 20))
    dX, dW, dY = to_device(X), to_device(W), to_device(Y0)
    rc = g.conv2d_im2row(p.dtype, shape_of(p), p.alpha, dX.data_ptr(), dW.data_ptr(), W.ld, p.beta, dY.data_ptr(), Y0.ld,
                         torch.cuda.current_stream().cuda_stream)
    assert rc == 0, g.gemm_status_string(rc)
    cfg = g.gemm_last_config()
    assert g.gemm_poll_status() == 0, hex(g.gemm_status_detail())
    from workloads import Matrix
    Y = Matrix(dY.cpu().numpy(), Y0.rows, Y0.cols, Y0.ld, DTYPE_F32)
    assert Y.padding_intact()
    bits = lambda x: x.view(np.uint32 if x.dtype.itemsize == 4 else np.uint16)
    assert np.array_equal(bits(dX.cpu().numpy()), bits(X.buf)) and np.array_equal(bits(dW.cpu().numpy()), bits(W.buf))
    return Y, cfg


def check(p, X, W, Y0, Y, integer=False):
    ref = oracle.conv2d_direct(p.dtype, geom_of(p), p.alpha, X.buf, W.buf, W.ld, p.beta, Y0.buf, Y0.ld)
    got = Y.window().astype(np.float64)
    if integer:
        assert np.array_equal(got, ref), "integer-valued layer is not bit-exact"
        return
    k = p.gemm_mnk[2]
    if p.dtype == DTYPE_F32:
        tol = oracle.fp32_tolerance(k, p.alpha, p.beta, X.max_abs(), W.max_abs(), Y0.max_abs() if p.beta != 0 else 0.0)
        err = float(np.max(np.abs(got - ref)))
        assert err <= tol, f"max |Y - Y_ref| = {err:.3e} > {tol:.3e}"
    else:
        rel = float(np.linalg.norm(got - ref) / np.linalg.norm(ref))
        assert rel <= 1e-3, f"relative Frobenius error {rel:.3e} > 1e-3"


def expected_route(p, W):
    if p.kh == 1 and p.stride == 1 and p.pad == 0:
        return g.CONV_LOWERING_IDENTITY
    # 16-bit layers are fused when TMA can fetch both operands: whole 64-channel chunks, and a filter matrix whose
    # columns start on 16-byte boundaries
    if p.dtype == DTYPE_F32:
        # with room in the workspace, layers that would need scalar loads through the index map are lowered first
        return g.CONV_LOWERING_FUSED if p.c_in % 4 == 0 else g.CONV_LOWERING_EXPLICIT
    if p.c_in % 64 == 0 and W.ld % 8 == 0:
        return g.CONV_LOWERING_FUSED
    return g.CONV_LOWERING_EXPLICIT


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_F16, DTYPE_BF16])
@pytest.mark.parametrize("gm", SMALL)
def test_layers_match_the_definition(gm, dtype):
    for (alpha, beta), ld_pad in (((1.0, 0.0), (0, 0)), ((1.5, 0.5), (8, 4))):
        p = make(gm, dtype, alpha=alpha, beta=beta, ld_pad=ld_pad)
        X, W, Y0 = p.operands()
        Y, cfg = run_conv(p, X, W, Y0)
        assert cfg["lowering"] == expected_route(p, W), cfg
        check(p, X, W, Y0, Y)
        p = make(gm, dtype, kind="int", alpha=alpha, beta=beta, ld_pad=ld_pad)
        X, W, Y0 = p.operands()
        Y, cfg = run_conv(p, X, W, Y0)
        check(p, X, W, Y0, Y, integer=True)


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_BF16])
@pytest.mark.parametrize("gm", SMALL)
def test_explicit_lowering_route(gm, dtype):
    g.conv2d_force_lowering(g.CONV_LOWERING_EXPLICIT)
    p = make(gm, dtype, kind="int", alpha=1.5, beta=0.5)
    X, W, Y0 = p.operands()
    Y, cfg = run_conv(p, X, W, Y0)
    assert cfg["lowering"] in (g.CONV_LOWERING_EXPLICIT, g.CONV_LOWERING_IDENTITY)
    check(p, X, W, Y0, Y, integer=True)


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_F16])
@pytest.mark.parametrize("gm", SMALL)
def test_im2row_kernel_writes_the_lowered_matrix_bit_for_bit(gm, dtype):
    p = make(gm, dtype)
    X, _, _ = p.operands()
    m, n, k = p.gemm_mnk
    for ld in (k, k + 3, (k + 7) // 8 * 8):
        want = oracle.im2row(dtype, geom_of(p), X.buf, ld=ld).reshape(n, ld)[:, :k]
        dX = to_device(X)
        out = torch.zeros(n * ld, dtype=dX.dtype, device="cuda")
        rc = g.im2row(dtype, shape_of(p), dX.data_ptr(), out.data_ptr(), ld, torch.cuda.current_stream().cuda_stream)
        assert rc == 0
        got = out.cpu().numpy().reshape(n, ld)[:, :k]
        bits = lambda x: np.ascontiguousarray(x).view(np.uint32 if x.dtype.itemsize == 4 else np.uint16)
        assert np.array_equal(bits(got), bits(want))


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_every_tensor_tile_with_the_im2col_producer(dtype):
    ensure_workspace(256 << 20)
    gm = (4, 19, 23, 128, 304, 3, 3, 1, 1)         # 1748 pixels, k = 1152
    for tile in ((128, 64), (128, 128), (128, 256), (256, 256)):
        for split in (1, 3):
            g.gemm_force_tile(tile[0], tile[1], split)
            p = make(gm, dtype, kind="int", alpha=1.0, beta=1.0)
            X, W, Y0 = p.operands()
            Y, cfg = run_conv(p, X, W, Y0)
            assert cfg["lowering"] == g.CONV_LOWERING_FUSED and cfg["kernel"] == g.GEMM_KERNEL_TENSOR
            assert (cfg["tile_m"], cfg["tile_n"]) == tile and cfg["split_k"] == split, cfg
            check(p, X, W, Y0, Y, integer=True)


def test_every_fp32_tile_with_the_index_map():
    ensure_workspace(256 << 20)
    for gm in ((2, 14, 15, 16, 200, 3, 3, 1, 1), (2, 14, 15, 6, 200, 3, 3, 2, 1)):      # 128-bit and scalar loads
        g.conv2d_force_lowering(g.CONV_LOWERING_FUSED)      # the scalar index map is otherwise taken only without a workspace
        for tile in ((128, 128), (128, 64), (64, 128), (64, 64)):
            for split in (1, 2):
                g.gemm_force_tile(tile[0], tile[1], split)
                p = make(gm, DTYPE_F32, kind="int", alpha=1.0, beta=1.0)
                X, W, Y0 = p.operands()
                Y, cfg = run_conv(p, X, W, Y0)
                assert cfg["lowering"] == g.CONV_LOWERING_FUSED and cfg["kernel"] == g.GEMM_KERNEL_SIMT_FAST
                assert (cfg["tile_m"], cfg["tile_n"]) == tile and cfg["vector_b"] == (4 if gm[3] % 4 == 0 else 1), cfg
                check(p, X, W, Y0, Y, integer=True)


def test_fp32_layer_with_three_channels_stays_fused_without_workspace():
    drop_workspace()
    p = make(SMALL[0], DTYPE_F32, alpha=1.5, beta=0.5)
    X, W, Y0 = p.operands()
    dX, dW, dY = to_device(X), to_device(W), to_device(Y0)
    rc = g.conv2d_im2row(p.dtype, shape_of(p), p.alpha, dX.data_ptr(), dW.data_ptr(), W.ld, p.beta, dY.data_ptr(), Y0.ld, 0)
    assert rc == 0 and g.gemm_poll_status() == 0
    assert g.gemm_last_config()["lowering"] == g.CONV_LOWERING_FUSED and g.gemm_last_config()["vector_b"] == 1
    from workloads import Matrix
    check(p, X, W, Y0, Matrix(dY.cpu().numpy(), Y0.rows, Y0.cols, Y0.ld, DTYPE_F32))


def test_sixteen_bit_layer_without_workspace_reports_it():
    drop_workspace()
    p = make(SMALL[0], DTYPE_BF16)
    X, W, Y0 = p.operands()
    dX, dW, dY = to_device(X), to_device(W), to_device(Y0)
    rc = g.conv2d_im2row(p.dtype, shape_of(p), 1.0, dX.data_ptr(), dW.data_ptr(), W.ld, 0.0, dY.data_ptr(), Y0.ld, 0)
    assert rc == g.GEMM_ERR_WORKSPACE
    assert np.array_equal(dY.cpu().numpy().view(np.uint32), Y0.buf.view(np.uint32))       # nothing written


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_BF16])
def test_activations_off_a_sixteen_byte_boundary(dtype):
    # X one element past an aligned address: no 128-bit loads, no TMA; with and without room for the lowered matrix
    gm = (2, 11, 9, 64, 48, 3, 3, 1, 1)
    p = make(gm, dtype, kind="int", alpha=1.0, beta=1.0)
    X, W, Y0 = p.operands()
    dX = to_device(X)
    shifted = torch.empty(dX.numel() + 1, dtype=dX.dtype, device="cuda")
    shifted[1:] = dX
    es = 4 if dtype == DTYPE_F32 else 2
    from workloads import Matrix
    for room in (True, False):
        if room:
            ensure_workspace(64 << 20)
        else:
            drop_workspace()
        dW, dY = to_device(W), to_device(Y0)
        rc = g.conv2d_im2row(dtype, shape_of(p), 1.0, shifted.data_ptr() + es, dW.data_ptr(), W.ld, 1.0, dY.data_ptr(), Y0.ld, 0)
        if dtype == DTYPE_BF16 and not room:
            assert rc == g.GEMM_ERR_WORKSPACE          # a 16-bit layer that TMA cannot lower needs the workspace
            continue
        assert rc == 0 and g.gemm_poll_status() == 0
        want = g.CONV_LOWERING_EXPLICIT if room else g.CONV_LOWERING_FUSED
        assert g.gemm_last_config()["lowering"] == want
        check(p, X, W, Y0, Matrix(dY.cpu().numpy(), Y0.rows, Y0.cols, Y0.ld, DTYPE_F32), integer=True)


def test_scaling_only_layer_call():
    # alpha == 0: Y <- beta*Y, activations and filters are not read (and may be null)
    p = make(SMALL[4], DTYPE_F32, alpha=0.0, beta=0.5, ld_pad=(0, 4))
    X, W, Y0 = p.operands()
    dY = to_device(Y0)
    rc = g.conv2d_im2row(p.dtype, shape_of(p), 0.0, 0, 0, W.ld, 0.5, dY.data_ptr(), Y0.ld, 0)
    assert rc == 0 and g.gemm_poll_status() == 0
    from workloads import Matrix
    Y = Matrix(dY.cpu().numpy(), Y0.rows, Y0.cols, Y0.ld, DTYPE_F32)
    assert Y.padding_intact() and np.array_equal(Y.window(), 0.5 * Y0.window())


def test_invalid_arguments():
    s = g.conv_shape(1, 4, 4, 4, 4, 5, 5, 1, 1, 0, 0)              # filter larger than the padded image
    assert g.conv2d_im2row(DTYPE_F32, s, 1.0, 16, 16, 4, 0.0, 16, 4, 0) == -2
    s = g.conv_shape(1, 4, 4, 4, 4, 3, 3, 1, 1, 1, 1)
    assert g.conv2d_im2row(7, s, 1.0, 16, 16, 4, 0.0, 16, 4, 0) == -1
    assert g.conv2d_im2row(DTYPE_F32, s, 1.0, 0, 16, 4, 0.0, 16, 4, 0) == -4
    assert g.conv2d_im2row(DTYPE_F32, s, 1.0, 16, 16, 3, 0.0, 16, 4, 0) == -6
    assert g.conv2d_im2row(DTYPE_F32, s, 1.0, 16, 16, 4, 0.0, 16, 3, 0) == -9


def sampled_check(p, X, W, Y0, Y, seed=0):
    rng = np.random.default_rng(seed)
    m, n, k = p.gemm_mnk
    rows = np.concatenate([[0, m - 1, 0, m - 1], rng.integers(0, m, 6000)])
    cols = np.concatenate([[0, n - 1, n - 1, 0], rng.integers(0, n, 6000)])
    ref = oracle.conv2d_samples_f64(p.dtype, geom_of(p), p.alpha, X.buf, W.buf, W.ld, p.beta, Y0.buf, Y0.ld, rows, cols)
    got = Y.window()[rows, cols].astype(np.float64)
    if p.kindX == "int":
        assert np.array_equal(got, ref)
    elif p.dtype == DTYPE_F32:
        tol = oracle.fp32_tolerance(k, p.alpha, p.beta, X.max_abs(), W.max_abs(), 0.0)
        assert float(np.max(np.abs(got - ref))) <= tol
    else:
        assert float(np.linalg.norm(got - ref) / np.linalg.norm(ref)) <= 1e-3


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_BF16])
def test_full_size_layers_on_sampled_entries(dtype):
    # batch 32, in the configuration the selector picks (the one the benchmark times): the 7 x 7 stem, 3 x 3 layers
    # of both networks and a 1 x 1 layer; entries at the corners and thousands of scattered ones against fp64
    rn, vg = conv_layer_problems("resnet50", dtype=dtype), conv_layer_problems("vgg16", dtype=dtype)
    rn_i = conv_layer_problems("resnet50", dtype=dtype, integer=True)
    for i, p in enumerate([rn[0], rn[2], rn[6], rn[16], rn[3], vg[0], vg[3], rn_i[11], rn_i[2]]):
        X, W, Y0 = p.operands()
        Y, cfg = run_conv(p, X, W, Y0)
        assert cfg["lowering"] == expected_route(p, W), (p.name, cfg)
        sampled_check(p, X, W, Y0, Y, seed=i)
