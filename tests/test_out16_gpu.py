"""Parity of the all-16-bit data types (GEMM_F16_C16, GEMM_BF16_C16: A, B and C in one 16-bit type, fp32
accumulation, one rounding at the store) with the CPU oracle, through the C ABI: every kernel that can write C
(tensor kernels with TMA and with direct stores, CTA pairs, split-k reduction, the generic kernel, the scaling-only
path), gemm_host, and the convolution front end.

Tolerance.  The library rounds an fp32 value r = alpha*acc + beta*C0 once, to nearest even, to the 16-bit type.  r
itself is within the tolerance of the fp32-result path of the exact value ref (for the tensor path: the relative
Frobenius bound 1e-3, which the entries here satisfy far more tightly because k is small), so
    |C - ref| <= ulp16(ref)/2 + slack,   slack = 4*2^-24*(k*|alpha|*max|A|*max|B| + |beta|*max|C0|) + ulp16(ref)/64,
where the last term covers results that fp32 rounding moves across a rounding boundary of the 16-bit type.
Integer-valued cases whose results are representable in the 16-bit type must be bit-exact."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import paper_2310_17408_b200 as g
from workloads import DTYPE_BF16, DTYPE_F16, ConvProblem, Matrix, Problem, make_matrix

from gpu_util import ensure_workspace, to_device

pytestmark = pytest.mark.gpu

OUT = {DTYPE_F16: g.GEMM_F16_C16, DTYPE_BF16: g.GEMM_BF16_C16}
PREC = {DTYPE_F16: 11, DTYPE_BF16: 8}          # significand bits of the result type
TRANS = list(itertools.product("NT", "NT"))


@pytest.fixture(autouse=True)
def _reset():
    yield
    g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
    g.gemm_force_tile(0, 0, 0)
    g.conv2d_force_lowering(0)


def ulp16(x, dtype):
    """Spacing of the 16-bit type around |x| (normal range; binary16 subnormal spacing below 2^-14)."""
    ax = np.maximum(np.abs(x), 2.0 ** -14 if dtype == DTYPE_F16 else 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(ax)) - (PREC[dtype] - 1))


def c0_16(p, dtype, kind):
    """The previous contents of C in the 16-bit type (generated like any other operand)."""
    return make_matrix(p.m, p.n, kind=kind, seed=p.seed, matrix_id=2, dtype=dtype, ld=max(1, p.m) + p.pad[2])


def run(p, dtype, A, B, C0, host=False):
    ensure_workspace(g.gemm_workspace_bytes(OUT[dtype], p.transA, p.transB, p.m, p.n, p.k) + (64 << 20))
    s = torch.cuda.current_stream().cuda_stream
    if host:
        hA, hB, hC = (torch.from_numpy(x.buf.view(np.int16).copy()).pin_memory() for x in (A, B, C0))
        rc = g.gemm_host(OUT[dtype], p.transA, p.transB, p.m, p.n, p.k, p.alpha, hA.data_ptr(), A.ld, hB.data_ptr(), B.ld,
                         p.beta, hC.data_ptr(), C0.ld, s)
        out = hC.numpy().view(np.uint16)
    else:
        dA, dB, dC = to_device(A), to_device(B), to_device(C0)
        rc = g.gemm(OUT[dtype], p.transA, p.transB, p.m, p.n, p.k, p.alpha, dA.data_ptr(), A.ld, dB.data_ptr(), B.ld, p.beta,
                    dC.data_ptr(), C0.ld, s)
        out = dC.cpu().numpy().view(np.uint16)
    assert rc == 0, g.gemm_status_string(rc)
    cfg = g.gemm_last_config()
    assert g.gemm_poll_status() == 0, hex(g.gemm_status_detail())
    C = Matrix(out.copy(), p.m, p.n, C0.ld, dtype)
    assert C.padding_intact(), "rows m..ldc-1 of C were written"
    return C, cfg


def check(p, dtype, A, B, C0, C, exact=False):
    # the oracle reads C0 as fp32: hand it the decoded 16-bit values
    c0f = np.zeros(C0.ld * p.n, dtype=np.float32)
    c0f.reshape(p.n, C0.ld).T[: p.m, :] = C0.as_f64().astype(np.float32)
    ref = oracle.gemm_l0(dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, A.buf, A.ld, B.buf, B.ld, p.beta, c0f, C0.ld,
                         acc=oracle.ACC_F64)
    got = C.as_f64()
    if exact:
        assert np.array_equal(got, ref), "representable integer results are not bit-exact"
        return
    u = ulp16(ref, dtype)
    slack = oracle.fp32_tolerance(p.k, p.alpha, p.beta, A.max_abs(), B.max_abs(), C0.max_abs() if p.beta != 0 else 0.0) + u / 64
    bad = np.abs(got - ref) > u / 2 + slack
    assert not bad.any(), f"{int(bad.sum())} entries off by more than half an ulp of the result type (+ fp32 slack)"


def problem(dtype, m, n, k, ta, tb, alpha, beta, kind, pad, seed=3):
    return Problem("t", dtype, m, n, k, alpha, beta, ta, tb, kindA=kind, kindB=kind, kindC=kind, seed=seed, pad=pad)


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
@pytest.mark.parametrize("ta,tb", TRANS)
def test_parity_grid(dtype, ta, tb):
    shapes = [(1, 1, 1), (64, 64, 64), (129, 257, 65), (200, 300, 150), (5, 1000, 33), (384, 520, 256), (130, 70, 17)]
    for family in (g.GEMM_KERNEL_SIMT_GENERIC, g.GEMM_KERNEL_TENSOR):
        g.gemm_force_kernel(family)
        for (m, n, k) in shapes:
            # pad 8 keeps C addressable by TMA tile stores (16-byte column stride), pad 3 forces direct stores
            for (alpha, beta), pad in (((1.0, 0.0), (0, 0, 0)), ((1.5, 0.5), (8, 8, 8)), ((-0.75, 1.0), (1, 3, 3))):
                p = problem(dtype, m, n, k, ta, tb, alpha, beta, "normal", pad, seed=m + n + k)
                A, B, _ = p.operands()
                C0 = c0_16(p, dtype, "normal")
                C, cfg = run(p, dtype, A, B, C0)
                check(p, dtype, A, B, C0, C)
            # integers in [-4, 4], k <= 16: |result| <= 16*16 + 4 is representable in both types
            kk = min(k, 16 if dtype == DTYPE_F16 else 12)
            p = problem(dtype, m, n, kk, ta, tb, 1.0, 1.0, "int", (0, 8, 0), seed=7 + m)
            A, B, _ = p.operands()
            C0 = c0_16(p, dtype, "int")
            C, cfg = run(p, dtype, A, B, C0)
            check(p, dtype, A, B, C0, C, exact=True)


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_every_tile_split_k_and_pairs(dtype):
    ensure_workspace(256 << 20)
    for (tm, tn), split in itertools.product([(128, 256), (128, 128), (128, 64), (256, 256)], (1, 3)):
        g.gemm_force_tile(tm, tn, split)
        for ta, tb in (("N", "N"), ("T", "T")):
            p = problem(dtype, 300, 520, 777, ta, tb, 1.5, 0.5, "normal", (0, 8, 4), seed=tm + tn + split)
            A, B, _ = p.operands()
            C0 = c0_16(p, dtype, "normal")
            C, cfg = run(p, dtype, A, B, C0)
            assert (cfg["kernel"], cfg["tile_m"], cfg["tile_n"]) == (g.GEMM_KERNEL_TENSOR, tm, tn), cfg
            assert cfg["split_k"] == split, cfg
            check(p, dtype, A, B, C0, C)


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_scaling_only_and_beta_zero_with_nan(dtype):
    p = problem(dtype, 70, 50, 40, "N", "N", 0.0, 0.5, "normal", (0, 0, 2))
    A, B, _ = p.operands()
    C0 = c0_16(p, dtype, "normal")
    C, cfg = run(p, dtype, A, B, C0)                 # alpha == 0: C <- beta*C, one rounding
    assert cfg["kernel"] == g.GEMM_KERNEL_SCALE_ONLY
    check(p, dtype, A, B, C0, C)
    p = problem(dtype, 70, 50, 40, "N", "N", 1.0, 0.0, "normal", (0, 0, 2))
    C0.buf.reshape(p.n, C0.ld).T[: p.m, :] = 0x7E00 if dtype == DTYPE_F16 else 0x7FC0      # NaN: must not be read
    C, _ = run(p, dtype, A, B, C0)
    assert np.all(np.isfinite(C.as_f64()))
    check(p, dtype, A, B, C0, C)


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_gemm_host_moves_sixteen_bit_results(dtype):
    p = problem(dtype, 1100, 2600, 300, "N", "N", 1.5, 0.5, "normal", (0, 0, 4))
    A, B, _ = p.operands()
    C0 = c0_16(p, dtype, "normal")
    C, _ = run(p, dtype, A, B, C0, host=True)
    check(p, dtype, A, B, C0, C)


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_convolution_layers_with_sixteen_bit_results(dtype):
    # one layer per lowering route: TMA im2col (C_in = 64), explicit im2row pass (C_in = 3), identity (1 x 1)
    for gm in ((2, 13, 11, 64, 96, 3, 3, 1, 1), (2, 9, 10, 3, 40, 3, 3, 2, 1), (3, 5, 5, 8, 24, 1, 1, 1, 0)):
        b, h, w, ci, co, kh, kw, st, pd = gm
        p = ConvProblem("t", dtype, b, h, w, ci, co, kh, kw, st, pd, 1.5, 0.5, seed=9, ld_pad=(0, 8))
        X, W, _ = p.operands()
        m, n, k = p.gemm_mnk
        Y0 = make_matrix(m, n, kind="normal", seed=9, matrix_id=2, dtype=dtype, ld=m + 8)
        shape = g.conv_shape(b, h, w, ci, co, kh, kw, st, st, pd, pd)
        ensure_workspace(g.conv2d_workspace_bytes(OUT[dtype], shape) + (64 << 20))
        dX, dW, dY = to_device(X), to_device(W), to_device(Y0)
        rc = g.conv2d_im2row(OUT[dtype], shape, p.alpha, dX.data_ptr(), dW.data_ptr(), W.ld, p.beta, dY.data_ptr(), Y0.ld,
                             torch.cuda.current_stream().cuda_stream)
        assert rc == 0 and g.gemm_poll_status() == 0
        Y = Matrix(dY.cpu().numpy().view(np.uint16).copy(), m, n, Y0.ld, dtype)
        assert Y.padding_intact()
        y0f = np.zeros(Y0.ld * n, dtype=np.float32)
        y0f.reshape(n, Y0.ld).T[:m, :] = Y0.as_f64().astype(np.float32)
        geo = oracle.conv_geom(b, h, w, ci, co, kh, kw, st, st, pd, pd)
        ref = oracle.conv2d_direct(dtype, geo, p.alpha, X.buf, W.buf, W.ld, p.beta, y0f, Y0.ld)
        u = ulp16(ref, dtype)
        slack = oracle.fp32_tolerance(k, p.alpha, p.beta, X.max_abs(), W.max_abs(), Y0.max_abs()) + u / 64
        assert not (np.abs(Y.as_f64() - ref) > u / 2 + slack).any()


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_strided_batch_with_sixteen_bit_results_on_the_tensor_cores(dtype):
    # a strided batch whose results are 16-bit as well: one launch of the tensor kernel, every problem's C found by its
    # byte offset; ragged shapes, C with padded leading dimension and a gap between the problems
    for (m, n, k), ta, tb, alpha, beta in [((72, 200, 136), "N", "N", 1.0, 0.0), ((130, 70, 264), "T", "N", 1.5, 0.5),
                                           ((64, 64, 64), "N", "T", -1.0, 1.0)]:
        batch, gap_c = 40, 5
        probs, As, Bs, Cs = [], [], [], []
        for b in range(batch):
            p = problem(dtype, m, n, k, ta, tb, alpha, beta, "normal", ((-(m if ta == "N" else k)) % 8, (-(k if tb == "N" else n)) % 8, 3), seed=40 + b)
            A, B, _ = p.operands()
            probs.append(p); As.append(A); Bs.append(B); Cs.append(c0_16(p, dtype, "normal"))
        sA, sB, sC = As[0].buf.size, Bs[0].buf.size, Cs[0].buf.size + gap_c
        assert sA % 8 == 0 and sB % 8 == 0
        hA = np.concatenate([a.buf for a in As]); hB = np.concatenate([b.buf for b in Bs])
        hC = np.zeros(sC * batch, dtype=np.uint16)
        for b in range(batch):
            hC[b * sC: b * sC + Cs[b].buf.size] = Cs[b].buf
        dev = lambda x: torch.from_numpy(x.view(np.int16)).cuda()
        dA, dB, dC = dev(hA), dev(hB), dev(hC)
        rc = g.gemm_strided_batched(OUT[dtype], ta, tb, m, n, k, alpha, dA.data_ptr(), As[0].ld, sA, dB.data_ptr(), Bs[0].ld, sB,
                                    beta, dC.data_ptr(), Cs[0].ld, sC, batch, torch.cuda.current_stream().cuda_stream)
        assert rc == 0, g.gemm_status_string(rc)
        cfg = g.gemm_last_config()
        assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["launches"] == 1, cfg
        assert g.gemm_poll_status() == 0, hex(g.gemm_status_detail())
        out = dC.cpu().numpy().view(np.uint16)
        for b in range(batch):
            C = Matrix(out[b * sC: b * sC + Cs[b].buf.size].copy(), m, n, Cs[b].ld, dtype)
            assert C.padding_intact()
            assert np.all(out[b * sC + Cs[b].buf.size: (b + 1) * sC] == 0)      # the gap keeps its zeros
            check(probs[b], dtype, As[b], Bs[b], Cs[b], C)
