"""Split k on the tensor cores finished inside the kernel: the CTAs that hold the k ranges of one tile run as a
thread-block cluster, park their accumulators in shared memory and sum the tile through distributed shared memory.
Checked against the CPU oracle and, bit for bit, against the other way of finishing a split (partial sums in the
workspace, reduction pass): both add the ranges in increasing order and apply the same epilogue."""
import itertools

import numpy as np
import pytest

import paper_2310_17408_b200 as g
from workloads import DTYPE_BF16, DTYPE_F16, Problem

from gpu_util import check_against_oracle, drop_workspace, ensure_workspace, run_problem

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _reset_forcing():
    yield
    g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
    g.gemm_force_tile(0, 0, 0)
    g.gemm_force_reduction(0)


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
@pytest.mark.parametrize("ta,tb", list(itertools.product("NT", "NT")))
def test_cluster_sum_equals_reduction_pass_and_oracle(dtype, ta, tb):
    ensure_workspace(128 << 20)
    for (m, n, k), tile_n, splits, pad in [((512, 1568, 2048), 128, 4, (0, 0, 0)), ((300, 520, 1100), 256, 3, (8, 8, 3)),
                                           ((130, 60, 1030), 64, 8, (0, 8, 1)), ((256, 264, 640), 128, 2, (0, 0, 0))]:
        for kind, alpha, beta in [("normal", 1.5, 0.5), ("int", 1.0, 0.0)]:
            p = Problem("ck", dtype, m, n, k, alpha, beta, ta, tb, kindA=kind, kindB=kind, kindC=kind if kind == "int" else "uniform",
                        seed=m + k, pad=pad)
            A, B, C0 = p.operands()
            g.gemm_force_tile(128, tile_n, splits)
            g.gemm_force_reduction(2)
            C_cl, cfg = run_problem(p, A, B, C0)
            repacks = bin(cfg["repacked"]).count("1")       # leading dimensions TMA cannot address are copied first
            assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["split_k"] >= 2 and cfg["launches"] == 1 + repacks, cfg
            check_against_oracle(p, A, B, C0, C_cl, integer=(kind == "int"))
            g.gemm_force_reduction(1)
            C_ws, cfg_ws = run_problem(p, A, B, C0)
            assert cfg_ws["split_k"] == cfg["split_k"] and cfg_ws["launches"] == 2 + repacks, cfg_ws
            assert np.array_equal(C_cl.buf.view(np.uint32), C_ws.buf.view(np.uint32)), (m, n, k, tile_n, splits)
            g.gemm_force_reduction(0)


def test_cluster_sum_needs_no_workspace_and_is_what_the_selector_takes():
    # few tiles, long k: the selector splits k; without any workspace that is only possible inside the kernel
    drop_workspace()
    p = Problem("ck0", DTYPE_BF16, 512, 1568, 4608, 1.0, 0.0, kindA="normal", kindB="normal", seed=17)
    A, B, C0 = p.operands()
    C, cfg = run_problem(p, A, B, C0, workspace=False)
    assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["split_k"] >= 2 and cfg["launches"] == 1, cfg
    check_against_oracle(p, A, B, C0, C)
    # 16-bit result through the same path
    q = Problem("ck16", DTYPE_BF16, 512, 520, 2048, 1.0, 0.0, kindA="int", kindB="int", kindC="int", seed=18)
    A, B, C0 = q.operands()
    g.gemm_force_tile(128, 128, 4)
    g.gemm_force_reduction(2)
    import torch
    from gpu_util import to_device
    dA, dB = to_device(A), to_device(B)
    dC = torch.zeros(q.m * q.n, dtype=torch.bfloat16, device="cuda")
    rc = g.gemm(g.GEMM_BF16_C16, "N", "N", q.m, q.n, q.k, 0.125, dA.data_ptr(), A.ld, dB.data_ptr(), B.ld, 0.0, dC.data_ptr(), q.m,
                torch.cuda.current_stream().cuda_stream)
    assert rc == 0 and g.gemm_poll_status() == 0
    assert g.gemm_last_config()["launches"] == 1
    want = 0.125 * (A.as_f64() @ B.as_f64())                     # multiples of 1/8
    got = dC.float().cpu().numpy().reshape(q.n, q.m).T.astype(np.float64)
    # bfloat16 has 8 significant bits: multiples of 1/8 are exact up to 32, beyond that one rounding of at most 2^-9 relative
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-6)
    assert np.array_equal(got[np.abs(want) <= 16], want[np.abs(want) <= 16])
