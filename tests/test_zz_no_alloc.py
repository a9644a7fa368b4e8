"""gemm_f32_splitk_static: the split-k GEMM for callers that cannot allocate device memory (its partial sums
live in a fixed array inside the library).  Its output is compared, on two calls in a row, with that of the
ordinary gemm() entry point on the same inputs and with the CPU oracle; the second call uses other data and
another shape, so that anything the first call left in the shared array would show.  Further cases cover the
branches of the entry point (128-bit loads, a k too short to split, alpha = 0, integer data bit for bit) and
check that a call really allocates nothing."""
import numpy as np
import pytest
import torch

import oracle
import paper_2310_17408_b200 as g
from workloads import Problem

pytestmark = pytest.mark.gpu


def _device(mat):
    return torch.from_numpy(mat.buf).cuda()


def _window(t, m, n, ld):
    return t.cpu().numpy().reshape(n, ld)[:, :m].T


def _oracle_args(p, A, B, C0):
    return (0, p.transA, p.transB, p.m, p.n, p.k, p.alpha, A.buf, A.ld, B.buf, B.ld, p.beta, C0.buf, C0.ld)


def test_static_scratch_entry_matches_gemm_twice_in_a_row():
    stream = torch.cuda.current_stream().cuda_stream
    g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
    g.gemm_force_tile(0, 0, 0)
    ws = torch.empty(32 << 20, dtype=torch.uint8, device="cuda")        # for the ordinary entry point only
    assert g.gemm_set_workspace(ws.data_ptr(), ws.numel(), 0) == 0
    try:
        cases = [(200, 136, 4100, "N", "N", 1.5, 0.5, 8), (96, 260, 2049, "T", "N", -1.0, 0.0, 5)]
        for call, (m, n, k, ta, tb, alpha, beta, split) in enumerate(cases):
            p = Problem("noalloc", 0, m, n, k, alpha, beta, ta, tb, seed=40 + call, pad=(0, 4, 3))
            A, B, C0 = p.operands()
            dA, dB = _device(A), _device(B)
            c_ref, c_new = _device(C0), _device(C0)
            assert g.gemm(0, ta, tb, m, n, k, alpha, dA.data_ptr(), A.ld, dB.data_ptr(), B.ld, beta,
                          c_ref.data_ptr(), C0.ld, stream) == 0
            rc = g.gemm_f32_splitk_static(ta, tb, m, n, k, alpha, dA.data_ptr(), A.ld, dB.data_ptr(), B.ld, beta,
                                          c_new.data_ptr(), C0.ld, split, stream)
            assert rc == 0, rc
            cfg = g.gemm_last_config()
            assert cfg["split_k"] > 1 and cfg["launches"] == 2, cfg
            torch.cuda.synchronize()
            ref = c_ref.cpu().numpy().reshape(n, C0.ld)
            new = c_new.cpu().numpy().reshape(n, C0.ld)
            # padding rows (NaN canaries) untouched; results within the fp32 bound the other tests use
            assert np.array_equal(new[:, m:].view(np.uint32), C0.buf.reshape(n, C0.ld)[:, m:].view(np.uint32))
            tol = oracle.fp32_tolerance(k, alpha, beta, A.max_abs(), B.max_abs(), C0.max_abs())
            err = float(np.max(np.abs(new[:, :m].astype(np.float64) - ref[:, :m].astype(np.float64))))
            assert err <= tol, (call, err, tol)
            # and against the CPU oracle (fp64 accumulation): the same bound
            want = oracle.gemm_l1(*_oracle_args(p, A, B, C0), acc=oracle.ACC_F64)
            err = float(np.max(np.abs(new[:, :m].T.astype(np.float64) - want)))
            assert err <= tol, (call, err, tol)
    finally:
        g.gemm_set_workspace(0, 0, 0)


def test_static_scratch_entry_against_the_oracle_on_its_branches():
    stream = torch.cuda.current_stream().cuda_stream
    #        m    n    k     tA   tB   alpha beta split  kind       pad        what it exercises
    cases = [(128, 64, 4096, "N", "N", 1.0, 0.0, 16, "int", (0, 0, 0)),        # aligned: 128-bit loads; bit-exact
             (128, 64, 4096, "T", "T", 1.5, 0.5, 7, "int", (0, 0, 0)),         # both transposed; integers: bit-exact
             (72, 40, 2050, "N", "T", -0.5, 1.0, 64, "uniform", (4, 4, 4)),    # transB; ld multiples of 4, ragged edges
             (64, 64, 16, "N", "N", 2.0, 0.5, 4, "uniform", (0, 0, 0)),        # k of one slice: single pass, no scratch
             (33, 17, 300, "T", "N", 0.0, 0.5, 2, "uniform", (1, 1, 1))]       # alpha = 0: C <- beta*C
    for i, (m, n, k, ta, tb, alpha, beta, split, kind, pad) in enumerate(cases):
        p = Problem("noalloc_b", 0, m, n, k, alpha, beta, ta, tb, kindA=kind, kindB=kind, kindC=kind, seed=60 + i, pad=pad)
        A, B, C0 = p.operands()
        dA, dB, dC = _device(A), _device(B), _device(C0)
        if alpha == 0.0:      # A and B must not be read: poison them
            dA.fill_(float("nan")); dB.fill_(float("inf"))
        rc = g.gemm_f32_splitk_static(ta, tb, m, n, k, alpha, dA.data_ptr(), A.ld, dB.data_ptr(), B.ld, beta,
                                      dC.data_ptr(), C0.ld, split, stream)
        assert rc == 0, (i, rc)
        cfg = g.gemm_last_config()
        torch.cuda.synchronize()
        got = _window(dC, m, n, C0.ld)
        if alpha == 0.0:
            assert cfg["kernel"] == g.GEMM_KERNEL_SCALE_ONLY
            assert np.array_equal(got, (np.float32(beta) * C0.window()).astype(np.float32))
        elif kind == "int":
            want = oracle.gemm_l0(*_oracle_args(p, A, B, C0), acc=oracle.ACC_F32)
            assert np.array_equal(got.astype(np.float32).view(np.uint32), np.ascontiguousarray(want).view(np.uint32)), i
        else:
            if k <= 16:
                assert cfg["split_k"] == 1 and cfg["launches"] == 1, cfg
            want = oracle.gemm_l1(*_oracle_args(p, A, B, C0), acc=oracle.ACC_F64)
            tol = oracle.fp32_tolerance(k, alpha, beta, A.max_abs(), B.max_abs(), C0.max_abs())
            err = float(np.max(np.abs(got.astype(np.float64) - want)))
            assert err <= tol, (i, err, tol)
        full = dC.cpu().numpy().reshape(n, C0.ld)
        assert np.array_equal(full[:, m:].view(np.uint32), C0.buf.reshape(n, C0.ld)[:, m:].view(np.uint32))


def test_static_scratch_entry_allocates_nothing():
    stream = torch.cuda.current_stream().cuda_stream
    p = Problem("noalloc_c", 0, 96, 80, 1024, 1.0, 0.0, seed=70)
    A, B, C0 = p.operands()
    dA, dB, dC = _device(A), _device(B), _device(C0)

    def call():
        rc = g.gemm_f32_splitk_static("N", "N", p.m, p.n, p.k, 1.0, dA.data_ptr(), A.ld, dB.data_ptr(), B.ld, 0.0,
                                      dC.data_ptr(), C0.ld, 8, stream)
        assert rc == 0
    call()                      # the first call on a device looks up the array's address
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    held0 = torch.cuda.memory_allocated()
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert torch.cuda.memory_allocated() == held0      # nothing taken from the framework's allocator
    assert free1 == free0                              # nor from the driver: free device memory is unchanged


def test_static_scratch_entry_rejects_what_does_not_fit():
    x = torch.zeros(16, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    big = 2048          # 2 partitions x 2048 x 2048 x 4 bytes = 32 MiB, more than the fixed array holds
    rc = g.gemm_f32_splitk_static("N", "N", big, big, 64, 1.0, x.data_ptr(), big, x.data_ptr(), 64, 0.0, x.data_ptr(),
                                  big, 2, s)
    assert rc == g.GEMM_ERR_TOO_LARGE
    assert g.gemm_f32_splitk_static("N", "N", 8, 8, 64, 1.0, x.data_ptr(), 8, x.data_ptr(), 64, 0.0, x.data_ptr(), 8, 1, s) == -14
    assert g.gemm_f32_splitk_static("N", "N", 8, 8, 64, 1.0, 0, 8, x.data_ptr(), 64, 0.0, x.data_ptr(), 8, 4, s) == -7
    torch.cuda.synchronize()
    assert torch.all(x == 0)
