"""GEMM_F32_TC: fp32 operands multiplied on the tensor cores as three bfloat16 pieces each.  Not IEEE fp32 arithmetic,
so it is held to the same bound as the fp32 path against the fp64 oracle, and must still be exact on integer-valued
data (a small integer is its own first piece; the other pieces are zero)."""
import itertools

import numpy as np
import pytest

import oracle
import paper_2310_17408_b200 as g
from workloads import DTYPE_F32, Problem, config_problems

from gpu_util import check_against_oracle, check_large, drop_workspace, ensure_workspace, run_problem

pytestmark = pytest.mark.gpu
TC = g.GEMM_F32_TC


@pytest.fixture(autouse=True)
def _reset_forcing():
    yield
    g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
    g.gemm_force_tile(0, 0, 0)


@pytest.mark.parametrize("ta,tb", list(itertools.product("NT", "NT")))
def test_split_precision_against_the_fp64_oracle(ta, tb):
    for (m, n, k), pad in [((512, 512, 512), (0, 0, 0)), ((640, 520, 700), (1, 2, 3)), ((300, 1100, 1030), (4, 0, 4))]:
        for kind, alpha, beta in [("uniform", 1.0, 0.0), ("uniform", 1.5, 0.5), ("int", -1.0, 1.0)]:
            p = Problem("tc3", DTYPE_F32, m, n, k, alpha, beta, ta, tb, kindA=kind, kindB=kind,
                        kindC=kind if kind == "int" else "uniform", seed=m + k, pad=pad)
            A, B, C0 = p.operands()
            g.gemm_force_kernel(g.GEMM_KERNEL_TENSOR)      # these sizes are below what the selector sends to the tensor cores
            C, cfg = run_problem(p, A, B, C0, api_dtype=TC)
            g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
            assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["launches"] >= 8, cfg      # two splitting passes + six products
            check_against_oracle(p, A, B, C0, C, integer=(kind == "int"))


@pytest.mark.parametrize("ta,tb", list(itertools.product("NT", "NT")))
def test_split_precision_as_one_launch_on_cta_pairs(ta, tb):
    # enough 256 x 256 tiles for every CTA pair: the six piece products run as one multiplication whose k loop walks the
    # pieces (stored one after the other along k, k padded to a multiple of 64 with zeros); ragged k, m, n and padding
    for (m, n, k), pad in [((2350, 2400, 200), (0, 0, 0)), ((2305, 2562, 333), (3, 1, 2))]:
        for kind, alpha, beta in [("uniform", 1.5, 0.5), ("int", -1.0, 1.0), ("uniform", 1.0, 0.0)]:
            p = Problem("tc3p", DTYPE_F32, m, n, k, alpha, beta, ta, tb, kindA=kind, kindB=kind,
                        kindC=kind if kind == "int" else "uniform", seed=m + k, pad=pad)
            A, B, C0 = p.operands()
            g.gemm_force_kernel(g.GEMM_KERNEL_TENSOR)      # below the size the selector sends to the tensor cores
            C, cfg = run_problem(p, A, B, C0, api_dtype=TC)
            g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
            assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["launches"] == 3 and cfg["tile_m"] == 256, cfg
            check_against_oracle(p, A, B, C0, C, integer=(kind == "int"))


def test_split_precision_error_is_at_the_level_of_fp32_arithmetic():
    # the same problem through the exact fp32 kernel and through the three-piece path: both errors against the fp64
    # oracle are reported; the three-piece path must stay within a small multiple of the exact kernel's error
    p = Problem("tc3e", DTYPE_F32, 2048, 1024, 2048, 1.0, 0.0, seed=9)
    A, B, C0 = p.operands()
    ref = oracle.gemm_l1(DTYPE_F32, "N", "N", p.m, p.n, p.k, 1.0, A.buf, A.ld, B.buf, B.ld, 0.0, C0.buf, C0.ld, acc=oracle.ACC_F64)
    C_exact, _ = run_problem(p, A, B, C0)
    C_tc, cfg = run_problem(p, A, B, C0, api_dtype=TC)
    assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR
    e_exact = float(np.max(np.abs(C_exact.window().astype(np.float64) - ref)))
    e_tc = float(np.max(np.abs(C_tc.window().astype(np.float64) - ref)))
    tol = oracle.fp32_tolerance(p.k, 1.0, 0.0, A.max_abs(), B.max_abs(), 0.0)
    print(f"max abs error vs fp64: exact fp32 kernel {e_exact:.3e}, three bfloat16 pieces {e_tc:.3e}, bound {tol:.3e}")
    assert e_tc <= tol and e_tc <= 8.0 * max(e_exact, 2.0 ** -24)


def test_split_precision_falls_back_to_the_exact_kernel():
    # no workspace: the call runs as GEMM_F32; too small to gain: likewise
    p = Problem("tc3f", DTYPE_F32, 1536, 1600, 1700, 1.5, 0.5, seed=3)
    A, B, C0 = p.operands()
    drop_workspace()
    C, cfg = run_problem(p, A, B, C0, workspace=False, api_dtype=TC)
    assert cfg["kernel"] == g.GEMM_KERNEL_SIMT_FAST, cfg
    check_against_oracle(p, A, B, C0, C)
    ensure_workspace(64 << 20)
    q = Problem("tc3s", DTYPE_F32, 96, 200, 300, 1.0, 0.0, seed=4)
    A, B, C0 = q.operands()
    C, cfg = run_problem(q, A, B, C0, api_dtype=TC)
    assert cfg["kernel"] in (g.GEMM_KERNEL_SIMT_FAST, g.GEMM_KERNEL_SIMT_DIRECT), cfg
    check_against_oracle(q, A, B, C0, C)


def test_split_precision_full_size_square():
    import dataclasses
    p = dataclasses.replace(config_problems(2)[2], name="sq4096_tc")      # 4096^3, alpha = 1.5, beta = 0.5
    A, B, C0 = p.operands()
    C, cfg = run_problem(p, A, B, C0, check_inputs=False, api_dtype=TC)
    assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["launches"] == 3, cfg      # two splitting passes, one multiplication
    check_large(p, A, B, C0, C, cfg, seed=5)
