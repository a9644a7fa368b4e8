"""Seeded random sweep over data types, transpose flags, shapes around tile and alignment boundaries, padded leading
dimensions and scalars, each case checked against the CPU oracle with the tolerance of its data type.  The cases are
drawn from a fixed seed, so a failure names a reproducible case."""
import numpy as np
import pytest

import paper_2310_17408_b200 as g
from workloads import DTYPE_BF16, DTYPE_F16, DTYPE_F32, Problem

from gpu_util import check_against_oracle, ensure_workspace, run_problem
import test_out16_gpu as o16

pytestmark = pytest.mark.gpu

EDGES = [1, 2, 7, 8, 9, 31, 32, 33, 63, 64, 65, 127, 128, 129, 136, 200, 255, 256, 257, 264, 300, 384, 511, 513]


def draw_cases(seed, count):
    rng = np.random.default_rng(seed)
    cases = []
    for _ in range(count):
        api = int(rng.choice([DTYPE_F32, DTYPE_F16, DTYPE_BF16, g.GEMM_F16_C16, g.GEMM_BF16_C16]))
        m, n = int(rng.choice(EDGES)), int(rng.choice(EDGES))
        k = int(rng.choice([1, 5, 16, 63, 64, 65, 130, 256, 700, 1100]))
        ta, tb = str(rng.choice(["N", "T"])), str(rng.choice(["N", "T"]))
        alpha, beta = [(1.0, 0.0), (1.5, 0.5), (-1.0, 1.0), (0.25, -2.0)][int(rng.integers(0, 4))]
        pad = tuple(int(x) for x in rng.choice([0, 1, 3, 4, 8], 3))
        force = int(rng.choice([0, 0, 0, 1, 2]))            # mostly the selector; sometimes a forced split or the pair kernel
        cases.append((api, m, n, k, ta, tb, alpha, beta, pad, force))
    return cases


@pytest.mark.parametrize("chunk", range(6))
def test_random_cases(chunk):
    ensure_workspace(256 << 20)
    for i, (api, m, n, k, ta, tb, alpha, beta, pad, force) in enumerate(draw_cases(1234 + chunk, 30)):
        g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
        g.gemm_force_tile(0, 0, 0)
        if force == 1:
            g.gemm_force_tile(0, 0, 3)
        elif force == 2 and api != DTYPE_F32:
            g.gemm_force_tile(256, 256, 0)
        tag = f"case {chunk}/{i}: api={api} {ta}{tb} {m}x{n}x{k} alpha={alpha} beta={beta} pad={pad} force={force}"
        try:
            if api in (g.GEMM_F16_C16, g.GEMM_BF16_C16):
                dtype = DTYPE_F16 if api == g.GEMM_F16_C16 else DTYPE_BF16
                p = Problem("f", dtype, m, n, k, alpha, beta, ta, tb, kindA="normal", kindB="normal", seed=chunk * 100 + i, pad=pad)
                A, B, _ = p.operands()
                C0 = o16.c0_16(p, dtype, "normal")
                C, _ = o16.run(p, dtype, A, B, C0)
                o16.check(p, dtype, A, B, C0, C)
            else:
                kind = "uniform" if api == DTYPE_F32 else "normal"
                p = Problem("f", api, m, n, k, alpha, beta, ta, tb, kindA=kind, kindB=kind, kindC="uniform", seed=chunk * 100 + i, pad=pad)
                A, B, C0 = p.operands()
                C, _ = run_problem(p, A, B, C0)
                check_against_oracle(p, A, B, C0, C)
        except AssertionError as exc:
            raise AssertionError(f"{tag}: {exc}") from exc
        finally:
            g.gemm_force_tile(0, 0, 0)


@pytest.mark.parametrize("chunk", range(3))
def test_random_convolution_layers(chunk):
    import torch
    import oracle
    from workloads import ConvProblem, Matrix, make_matrix
    from gpu_util import to_device
    rng = np.random.default_rng(4321 + chunk)
    for i in range(25):
        api = int(rng.choice([DTYPE_F32, DTYPE_F16, DTYPE_BF16, g.GEMM_F16_C16, g.GEMM_BF16_C16]))
        dtype = {g.GEMM_F16_C16: DTYPE_F16, g.GEMM_BF16_C16: DTYPE_BF16}.get(api, api)
        c16 = api != dtype
        b, h, w = int(rng.integers(1, 4)), int(rng.integers(4, 21)), int(rng.integers(4, 21))
        ci, co = int(rng.choice([3, 4, 8, 16, 64, 128])), int(rng.choice([5, 8, 40, 64, 136]))
        ks = int(rng.choice([1, 3, 5]))
        st, pd = int(rng.integers(1, 3)), int(rng.integers(0, ks // 2 + 1))
        if h + 2 * pd < ks or w + 2 * pd < ks:
            continue
        alpha, beta = [(1.0, 0.0), (1.5, 0.5), (-1.0, 1.0)][int(rng.integers(0, 3))]
        p = ConvProblem("f", dtype, b, h, w, ci, co, ks, ks, st, pd, alpha, beta, seed=chunk * 100 + i,
                        ld_pad=(int(rng.choice([0, 8])), int(rng.choice([0, 3, 8]))))
        X, W, Y0f = p.operands()
        m, n, k = p.gemm_mnk
        Y0 = make_matrix(m, n, kind="normal", seed=p.seed, matrix_id=2, dtype=dtype, ld=Y0f.ld) if c16 else Y0f
        shape = g.conv_shape(b, h, w, ci, co, ks, ks, st, st, pd, pd)
        ensure_workspace(g.conv2d_workspace_bytes(api, shape) + (64 << 20))
        dX, dW, dY = to_device(X), to_device(W), to_device(Y0)
        rc = g.conv2d_im2row(api, shape, alpha, dX.data_ptr(), dW.data_ptr(), W.ld, beta, dY.data_ptr(), Y0.ld,
                             torch.cuda.current_stream().cuda_stream)
        tag = f"conv case {chunk}/{i}: api={api} {b}x{h}x{w}x{ci}->{co} k{ks} s{st} p{pd} alpha={alpha} beta={beta} ld={W.ld},{Y0.ld}"
        assert rc == 0 and g.gemm_poll_status() == 0, tag
        out = dY.cpu().numpy()
        Y = Matrix(out.view(np.uint16).copy() if c16 else out, m, n, Y0.ld, dtype if c16 else DTYPE_F32)
        assert Y.padding_intact(), tag
        y0f = np.zeros(Y0.ld * n, dtype=np.float32)
        y0f.reshape(n, Y0.ld).T[:m, :] = Y0.as_f64().astype(np.float32)
        geo = oracle.conv_geom(b, h, w, ci, co, ks, ks, st, st, pd, pd)
        ref = oracle.conv2d_direct(dtype, geo, alpha, X.buf, W.buf, W.ld, beta, y0f, Y0.ld)
        got = Y.as_f64()
        slack = oracle.fp32_tolerance(k, alpha, beta, X.max_abs(), W.max_abs(), Y0.max_abs() if beta != 0 else 0.0)
        if c16:
            u = o16.ulp16(ref, dtype)
            assert not (np.abs(got - ref) > u / 2 + slack + u / 64).any(), tag
        elif dtype == DTYPE_F32:
            assert float(np.max(np.abs(got - ref))) <= slack, tag
        else:
            assert float(np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)) <= 1e-3, tag


@pytest.mark.parametrize("chunk", range(3))
def test_random_cases_on_the_special_paths(chunk):
    """Shapes drawn where the selector leaves the common kernels: few rows and many columns (exchanged operand roles),
    few tiles and long k (split k summed by clusters, or by the separate pass when forced), tiny problems (the kernel
    without staging), fp32 data on the tensor cores in both of its forms, and host buffers through gemm_host."""
    import torch
    rng = np.random.default_rng(777 + chunk)
    ensure_workspace(512 << 20)
    for i in range(24):
        g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
        g.gemm_force_tile(0, 0, 0)
        g.gemm_force_reduction(0)
        what = str(rng.choice(["roles", "cluster", "tiny", "tc3", "tc3_one_launch", "host"]))
        ta, tb = str(rng.choice(["N", "T"])), str(rng.choice(["N", "T"]))
        alpha, beta = [(1.0, 0.0), (1.5, 0.5), (-1.0, 1.0), (0.25, -2.0)][int(rng.integers(0, 4))]
        pad = tuple(int(x) for x in rng.choice([0, 1, 3, 4, 8], 3))
        integer = bool(rng.integers(0, 3) == 0)
        api = None
        if what == "roles":
            dt = int(rng.choice([DTYPE_F16, DTYPE_BF16]))
            m, n, k = int(rng.integers(1, 65)), int(rng.integers(1024, 6000)), int(rng.choice([8, 27, 64, 147, 152, 256, 576, 1000]))
        elif what == "cluster":
            dt = int(rng.choice([DTYPE_F32, DTYPE_BF16]))
            m, n, k = int(rng.choice([64, 128, 200, 256, 512])), int(rng.choice([64, 128, 300, 512, 1568])), int(rng.choice([512, 1024, 2304, 4608]))
            if rng.integers(0, 2):
                g.gemm_force_reduction(int(rng.choice([1, 2])))
        elif what == "tiny":
            dt, (m, n, k) = DTYPE_F32, (int(rng.integers(1, 260)), int(rng.integers(1, 260)), int(rng.integers(1, 400)))
        elif what == "tc3":
            dt, api = DTYPE_F32, g.GEMM_F32_TC
            m, n, k = int(rng.integers(129, 900)), int(rng.integers(128, 900)), int(rng.integers(64, 1200))
            g.gemm_force_kernel(g.GEMM_KERNEL_TENSOR)
        elif what == "tc3_one_launch":
            dt, api = DTYPE_F32, g.GEMM_F32_TC
            m, n, k = int(rng.integers(1025, 2600)), int(rng.integers(1025, 2600)), int(rng.integers(64, 400))
            g.gemm_force_kernel(g.GEMM_KERNEL_TENSOR)
        else:
            dt = int(rng.choice([DTYPE_F32, DTYPE_BF16]))
            m, n, k = int(rng.integers(1, 700)), int(rng.integers(1, 3000)), int(rng.integers(0, 900))
        kind = "int" if integer else ("uniform" if dt == DTYPE_F32 else "normal")
        p = Problem("f", dt, m, n, k, alpha, beta, ta, tb, kindA=kind, kindB=kind, kindC="int" if integer else "uniform",
                    seed=chunk * 100 + i, pad=pad)
        tag = f"case {chunk}/{i}: {what} dtype={dt} {ta}{tb} {m}x{n}x{k} alpha={alpha} beta={beta} pad={pad} integer={integer}"
        A, B, C0 = p.operands()
        try:
            if what == "host":
                C = C0.copy()
                rc = g.gemm_host(dt, ta, tb, m, n, k, alpha, A.buf.ctypes.data, A.ld, B.buf.ctypes.data, B.ld, beta,
                                 C.buf.ctypes.data, C.ld, torch.cuda.current_stream().cuda_stream)
                assert rc == 0 and g.gemm_poll_status() == 0 and C.padding_intact()
            else:
                C, _ = run_problem(p, A, B, C0, api_dtype=api)
            check_against_oracle(p, A, B, C0, C, integer=integer)
        except AssertionError as exc:
            raise AssertionError(f"{tag}: {exc}") from exc
        finally:
            g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
            g.gemm_force_reduction(0)
