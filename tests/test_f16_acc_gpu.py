"""GEMM_F16_ACC16: binary16 inputs, binary16 accumulation on the tensor cores, binary16 result (the paper's f16
arithmetic, Section III-D), against the oracle's binary16 accumulation mode.

Tolerance.  The oracle rounds the running sum to binary16 after every product; the tensor core rounds it as its
hardware does (at the latest once per k block).  Either way each rounding moves the running sum by at most half a unit
in its last place, u = 2^-11 relative, so both results lie within k*u*S of the exact sum, S = sum_p |a_ip b_pj|, and
within 2*k*u*S of each other; alpha scales that, and the store adds half an ulp of the result.  Where every partial
sum is a binary16 number (small integers) nothing is ever rounded and the results must be identical."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import paper_2310_17408_b200 as g
from workloads import DTYPE_F16, make_matrix
from workloads.generators import decode_16

from gpu_util import ensure_workspace, to_device

pytestmark = pytest.mark.gpu
ACC16 = g.GEMM_F16_ACC16


@pytest.fixture(autouse=True)
def _reset_forcing():
    yield
    g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
    g.gemm_force_tile(0, 0, 0)


def run(m, n, k, ta, tb, alpha, beta, kind, seed, pad=(0, 0, 0), scale=1.0):
    (ar, ac), (br, bc) = ((m, k) if ta == "N" else (k, m)), ((k, n) if tb == "N" else (n, k))
    A = make_matrix(ar, ac, kind=kind, seed=seed, matrix_id=0, dtype=DTYPE_F16, ld=ar + pad[0], scale=scale)
    B = make_matrix(br, bc, kind=kind, seed=seed, matrix_id=1, dtype=DTYPE_F16, ld=br + pad[1], scale=scale)
    C0 = make_matrix(m, n, kind=kind if kind == "int" else "uniform", seed=seed, matrix_id=2, dtype=DTYPE_F16, ld=m + pad[2])
    ensure_workspace(64 << 20)
    dA, dB, dC = to_device(A), to_device(B), to_device(C0)
    rc = g.gemm(ACC16, ta, tb, m, n, k, alpha, dA.data_ptr(), A.ld, dB.data_ptr(), B.ld, beta, dC.data_ptr(), C0.ld,
                torch.cuda.current_stream().cuda_stream)
    assert rc == 0, g.gemm_status_string(rc)
    cfg = g.gemm_last_config()
    assert g.gemm_poll_status() == 0, hex(g.gemm_status_detail())
    out = dC.cpu().numpy().view(np.uint16).reshape(n, C0.ld)
    assert np.all(out[:, m:] == C0.buf.reshape(n, C0.ld)[:, m:]), "rows m..ldc-1 were written"
    got = decode_16(np.ascontiguousarray(out[:, :m].T), DTYPE_F16)
    c0 = C0.as_f64().astype(np.float32)                                   # the oracle reads C0 as fp32: every binary16 number is one
    c0_flat = np.ascontiguousarray(c0.T).ravel()
    want = oracle.gemm_l0(DTYPE_F16, ta, tb, m, n, k, alpha, A.buf, A.ld, B.buf, B.ld, beta, c0_flat, m, acc=oracle.ACC_F16)
    return got, want, (A, B, C0), cfg


@pytest.mark.parametrize("ta,tb", list(itertools.product("NT", "NT")))
def test_small_integers_are_exact(ta, tb):
    # entries in [-4, 4], k <= 128: every partial sum is an integer of magnitude <= 2048, a binary16 number
    for (m, n, k), pad in [((128, 64, 64), (0, 0, 0)), ((200, 300, 128), (8, 8, 1)), ((5, 1000, 33), (3, 0, 8)), ((384, 520, 100), (0, 8, 0))]:
        got, want, _, cfg = run(m, n, k, ta, tb, 1.0, 0.0, "int", seed=m + k, pad=pad)
        assert np.array_equal(got, want), (m, n, k, cfg)
        got, want, _, _ = run(m, n, k, ta, tb, 0.5, 1.0, "int", seed=m + k + 1, pad=pad)      # halves and small integers: exact too
        assert np.array_equal(got, np.array([[oracle.round_f16(v) for v in row] for row in want])), (m, n, k)


@pytest.mark.parametrize("tile_n", [0, 64, 128, 256])
def test_random_data_within_the_rounding_bound(tile_n):
    for (m, n, k), (ta, tb) in [((256, 512, 1024), ("N", "N")), ((300, 260, 2050), ("T", "N")), ((130, 700, 520), ("N", "T"))]:
        if tile_n:
            g.gemm_force_tile(128, tile_n, 1)
        alpha, beta = 1.5, 0.5
        got, want, (A, B, C0), cfg = run(m, n, k, ta, tb, alpha, beta, "normal", seed=k, scale=0.25)
        assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["split_k"] == 1, cfg
        a = np.abs(A.as_f64() if ta == "N" else A.as_f64().T)
        b = np.abs(B.as_f64() if tb == "N" else B.as_f64().T)
        S = a @ b                                                               # sum_p |a_ip b_pj|
        u = 2.0 ** -11
        bound = 2.0 * k * u * S * abs(alpha) + 2.0 * u * np.abs(want) + 2.0 ** -24
        err = np.abs(got - want)
        assert np.all(err <= bound), (float(np.max(err / bound)), cfg)
        # against the exact (fp64) result: inside the one-sided bound, and, somewhere, well above the single final
        # rounding that an fp32 accumulator would leave: the accumulation really is binary16
        exact = oracle.gemm_l0(DTYPE_F16, ta, tb, m, n, k, alpha, A.buf, A.ld, B.buf, B.ld, beta,
                               np.ascontiguousarray(C0.as_f64().astype(np.float32).T).ravel(), m, acc=oracle.ACC_F64)
        assert np.all(np.abs(got - exact) <= 0.5 * bound + 2.0 * u * np.abs(exact))
        assert np.max(np.abs(got - exact) / (u * np.abs(exact) + 2.0 ** -20)) > 4.0
        print(f"{m}x{n}x{k} tile_n={cfg['tile_n']}: max |gpu - oracle_f16| = {float(err.max()):.3e}, max |gpu - exact| = "
              f"{float(np.abs(got - exact).max()):.3e}, max |oracle_f16 - exact| = {float(np.abs(want - exact).max()):.3e}")


def test_overflow_and_degenerate_cases():
    # a sum beyond the binary16 range overflows to infinity, as in the oracle; alpha = 0 scales only; k = 0 likewise
    m, n, k = 128, 64, 64
    A = torch.full((k * m,), 60.0, device="cuda", dtype=torch.float16)
    B = torch.full((n * k,), 60.0, device="cuda", dtype=torch.float16)
    C = torch.zeros(m * n, device="cuda", dtype=torch.float16)
    s = torch.cuda.current_stream().cuda_stream
    assert g.gemm(ACC16, "N", "N", m, n, k, 1.0, A.data_ptr(), m, B.data_ptr(), k, 0.0, C.data_ptr(), m, s) == 0
    assert g.gemm_poll_status() == 0
    assert bool(torch.isinf(C).all())                                      # 64 * 3600 = 230400 > 65504
    C.fill_(3.0)
    assert g.gemm(ACC16, "N", "N", m, n, k, 0.0, 0, m, 0, k, 0.5, C.data_ptr(), m, s) == 0
    torch.cuda.synchronize()
    assert bool((C == 1.5).all())
