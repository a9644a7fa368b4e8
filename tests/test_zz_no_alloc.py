"""gemm_f32_splitk_static: the split-k GEMM for callers that cannot allocate device memory (its partial sums
live in a fixed array inside the library).  Its output is compared with that of the ordinary gemm() entry
point on the same inputs, on two calls in a row; the second call uses other data and another shape, so that
anything the first call left in the shared array would show."""
import numpy as np
import pytest
import torch

import oracle
import paper_2310_17408_b200 as g
from workloads import Problem

pytestmark = pytest.mark.gpu


def _device(mat):
    return torch.from_numpy(mat.buf).cuda()


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
            assert rc == 0, g.gemm_status_string(rc)
            torch.cuda.synchronize()
            ref = c_ref.cpu().numpy().reshape(n, C0.ld)
            new = c_new.cpu().numpy().reshape(n, C0.ld)
            # padding rows (NaN canaries) untouched; results within the fp32 bound the other tests use
            assert np.array_equal(new[:, m:].view(np.uint32), C0.buf.reshape(n, C0.ld)[:, m:].view(np.uint32))
            tol = oracle.fp32_tolerance(k, alpha, beta, A.max_abs(), B.max_abs(), C0.max_abs())
            err = float(np.max(np.abs(new[:, :m].astype(np.float64) - ref[:, :m].astype(np.float64))))
            assert err <= tol, (call, err, tol)
    finally:
        g.gemm_set_workspace(0, 0, 0)


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
