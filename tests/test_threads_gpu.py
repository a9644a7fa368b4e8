"""Concurrent callers: two host threads, each with its own stream and its own workspace registered for that stream,
run split-k configurations (which keep partial sums in the workspace) at the same time; every result is compared
with the CPU oracle.  With one shared workspace the partial sums of the two threads would overwrite each other."""
import threading

import numpy as np
import pytest
import torch

import oracle
import paper_2310_17408_b200 as g
from workloads import DTYPE_BF16, DTYPE_F32, Problem

from gpu_util import to_device

pytestmark = pytest.mark.gpu


def _worker(idx, dtype, shape, errors, rounds=12):
    try:
        torch.cuda.set_device(0)
        stream = torch.cuda.Stream()
        ws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
        assert g.gemm_set_workspace(ws.data_ptr(), ws.numel(), stream.cuda_stream) == 0
        m, n, k = shape
        p = Problem(f"thr{idx}", dtype, m, n, k, 1.5, 0.5, kindA="int", kindB="int", kindC="int", seed=500 + idx)
        A, B, C0 = p.operands()
        want = oracle.gemm_l1(dtype, "N", "N", m, n, k, p.alpha, A.buf, A.ld, B.buf, B.ld, p.beta, C0.buf, C0.ld,
                              acc=oracle.ACC_F32)        # integer data: exact in any order
        with torch.cuda.stream(stream):
            dA, dB = to_device(A), to_device(B)
            outs = [to_device(C0) for _ in range(rounds)]
            stream.synchronize()
            g.gemm_force_tile(0, 0, 4)          # acts on this thread only
            for dC in outs:
                rc = g.gemm(dtype, "N", "N", m, n, k, p.alpha, dA.data_ptr(), A.ld, dB.data_ptr(), B.ld, p.beta,
                            dC.data_ptr(), C0.ld, stream.cuda_stream)
                assert rc == 0, g.gemm_status_string(rc)
                cfg = g.gemm_last_config()
                assert cfg["split_k"] == 4, cfg
            stream.synchronize()
            for dC in outs:
                got = dC.cpu().numpy().reshape(n, C0.ld).T[:m]
                assert np.array_equal(got, want), f"thread {idx}: result differs from the oracle"
        assert g.gemm_set_workspace(0, 0, stream.cuda_stream) == 0
    except BaseException as exc:      # reported by the main thread
        errors.append((idx, repr(exc)))


def test_two_threads_two_streams_two_workspaces():
    errors = []
    threads = [threading.Thread(target=_worker, args=(0, DTYPE_F32, (256, 320, 4096), errors)),
               threading.Thread(target=_worker, args=(1, DTYPE_BF16, (512, 520, 4608), errors))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert g.gemm_poll_status() == 0, hex(g.gemm_status_detail())
    assert not errors, errors
    # the forcing of the worker threads did not leak into this one
    x = torch.zeros(64 * 64, device="cuda")
    assert g.gemm(DTYPE_F32, "N", "N", 64, 64, 64, 1.0, x.data_ptr(), 64, x.data_ptr(), 64, 0.0, x.data_ptr(), 64,
                  torch.cuda.current_stream().cuda_stream) == 0
    assert g.gemm_last_config()["split_k"] == 1
