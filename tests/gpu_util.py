"""Helpers for the GPU parity tests: run a workloads.Problem through the C ABI and compare with the oracle."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2310_17408_b200 as g
from workloads import DTYPE_F32, Matrix, Problem

_WS = {}


def ensure_workspace(nbytes: int):
    """Register a workspace of at least nbytes (kept alive here; the library does not own it)."""
    cur = _WS.get("t")
    if cur is None or cur.numel() < nbytes:
        _WS["t"] = torch.empty(max(nbytes, 1 << 20), dtype=torch.uint8, device="cuda")
        cur = _WS["t"]
    assert g.gemm_set_workspace(cur.data_ptr(), cur.numel(), 0) == 0


def drop_workspace():
    assert g.gemm_set_workspace(0, 0, 0) == 0
    _WS.pop("t", None)


def to_device(mat: Matrix) -> torch.Tensor:
    return torch.from_numpy(mat.buf.view(np.int16) if mat.buf.dtype == np.uint16 else mat.buf).cuda()


def run_problem(p: Problem, A: Matrix, B: Matrix, C0: Matrix, *, workspace=True, check_inputs=True, api_dtype=None):
    """Returns (C as Matrix on the host, config dict).  Asserts rc == 0, padding rows of C untouched,
    A and B unmodified, and the device status word clean.  api_dtype: the library's data-type code when it is not
    the element type of the operands (GEMM_F32_TC)."""
    code = p.dtype if api_dtype is None else api_dtype
    if workspace:
        ensure_workspace(g.gemm_workspace_bytes(code, p.transA, p.transB, p.m, p.n, p.k) + (64 << 20))
    dA, dB, dC = to_device(A), to_device(B), to_device(C0)
    rc = g.gemm(code, p.transA, p.transB, p.m, p.n, p.k, p.alpha, dA.data_ptr(), A.ld, dB.data_ptr(), B.ld,
                p.beta, dC.data_ptr(), C0.ld, torch.cuda.current_stream().cuda_stream)
    assert rc == 0, g.gemm_status_string(rc)
    cfg = g.gemm_last_config()
    assert g.gemm_poll_status() == 0, hex(g.gemm_status_detail())
    C = Matrix(dC.cpu().numpy(), p.m, p.n, C0.ld, DTYPE_F32)
    assert C.padding_intact(), "rows m..ldc-1 of C were written"
    if check_inputs:
        bits = lambda x: x.view(np.uint32 if x.dtype.itemsize == 4 else np.uint16)   # NaN canaries: compare bit patterns
        assert np.array_equal(bits(dA.cpu().numpy()), bits(A.buf)), "A was modified"
        assert np.array_equal(bits(dB.cpu().numpy()), bits(B.buf)), "B was modified"
    return C, cfg


def oracle_f64(p: Problem, A: Matrix, B: Matrix, C0: Matrix) -> np.ndarray:
    """fp64 truth of the whole result (blocked oracle in double: same values as the definition up to fp64 rounding)."""
    return oracle.gemm_l1(p.dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, A.buf, A.ld, B.buf, B.ld,
                          p.beta, C0.buf, C0.ld, acc=oracle.ACC_F64)


def fp32_tol(p: Problem, A: Matrix, B: Matrix, C0: Matrix) -> float:
    return oracle.fp32_tolerance(p.k, p.alpha, p.beta, A.max_abs(), B.max_abs(), C0.max_abs() if p.beta != 0 else 0.0)


def check_against_oracle(p: Problem, A: Matrix, B: Matrix, C0: Matrix, C: Matrix, *, integer=False):
    got = C.window()
    if integer:
        # every partial sum is an exactly representable integer multiple of 0.5: any summation order agrees bitwise
        want = oracle.gemm_l0(p.dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, A.buf, A.ld, B.buf, B.ld,
                              p.beta, C0.buf, C0.ld, acc=oracle.ACC_F32)
        # compared as values: equal bit for bit except that -0.0 and +0.0 count as equal.  The only place the two sides
        # can differ in the sign of a zero is the quick return for k = 0 or alpha = 0, where the library forms beta*C0 alone
        # (the BLAS convention: -2 * 0 = -0) and the definition adds alpha*0 to it (+0); NaN never compares equal.
        assert np.array_equal(np.ascontiguousarray(got), np.ascontiguousarray(want)), "integer-valued case is not bit-exact"
        return 0.0
    ref = oracle_f64(p, A, B, C0)
    if p.dtype == DTYPE_F32:
        err = float(np.max(np.abs(got.astype(np.float64) - ref))) if ref.size else 0.0
        tol = fp32_tol(p, A, B, C0)
        assert err <= tol, f"max |C - C_ref| = {err:.3e} > {tol:.3e}"
        return err
    num = np.linalg.norm(got.astype(np.float64) - ref)
    den = np.linalg.norm(ref)
    rel = float(num / den) if den > 0 else float(num)
    assert rel <= 1e-3, f"relative Frobenius error {rel:.3e} > 1e-3"
    return rel


def sample_positions(m, n, tile_m, tile_n, rng, scattered=4096):
    """Entries to verify one by one on large problems: corners, last row/column of distinct tile residues, random."""
    rows = [0, m - 1, 0, m - 1]
    cols = [0, n - 1, n - 1, 0]
    for i in {min(m - 1, tile_m - 1), min(m - 1, tile_m), m - 1, (m - 1) // tile_m * tile_m}:
        for j in {min(n - 1, tile_n - 1), min(n - 1, tile_n), n - 1, (n - 1) // tile_n * tile_n}:
            rows.append(i), cols.append(j)
    rows += list(rng.integers(0, m, scattered))
    cols += list(rng.integers(0, n, scattered))
    return np.array(rows, dtype=np.int64), np.array(cols, dtype=np.int64)


def check_large(p: Problem, A: Matrix, B: Matrix, C0: Matrix, C: Matrix, cfg, seed=0):
    """Whole-matrix randomised check plus exact fp64 values of sampled entries, full rows and full columns."""
    rng = np.random.default_rng(seed)
    m, n, k = p.m, p.n, p.k
    # (1) Freivalds: C x against alpha A (B x) + beta C0 x.  Each entry may be off by the per-entry bound; over a
    # row the n signed errors add up like a random walk, so the residual is judged against 4 sqrt(n) times it.
    tol_entry = fp32_tol(p, A, B, C0) * (1.0 if p.dtype == DTYPE_F32 else 2.0)
    for _ in range(4):
        x = rng.choice([-1.0, 1.0], n)
        resid, _ = oracle.freivalds(p.dtype, p.transA, p.transB, m, n, k, p.alpha, A.buf, A.ld, B.buf, B.ld,
                                    p.beta, C0.buf, C0.ld, C.buf, C.ld, x)
        bound = 4.0 * np.sqrt(n) * tol_entry
        worst = float(np.max(np.abs(resid)))
        assert worst <= bound, f"Freivalds residual {worst:.3e} > {bound:.3e}"
    # (2) sampled entries, 64 full rows and 64 full columns against exact fp64 dot products (rows and columns longer
    # than `line_cap` entries are sampled at that many random positions; the cap shrinks with k so that the CPU
    # work stays near 2^35 multiply-adds)
    rows, cols = sample_positions(m, n, cfg["tile_m"], cfg["tile_n"], rng)
    fr = rng.integers(0, m, 64)
    fc = rng.integers(0, n, 64)
    line_cap = int(max(512, min(8192, (1 << 35) // (128 * max(k, 1)))))
    nrow_samples = min(n, line_cap)
    for i in fr:
        js = rng.choice(n, nrow_samples, replace=False) if n > nrow_samples else np.arange(n)
        rows = np.concatenate([rows, np.full(js.size, i)]); cols = np.concatenate([cols, js])
    ncol_samples = min(m, line_cap)
    for j in fc:
        is_ = rng.choice(m, ncol_samples, replace=False) if m > ncol_samples else np.arange(m)
        rows = np.concatenate([rows, is_]); cols = np.concatenate([cols, np.full(is_.size, j)])
    ref = oracle.gemm_samples_f64(p.dtype, p.transA, p.transB, k, p.alpha, A.buf, A.ld, B.buf, B.ld, p.beta,
                                  C0.buf, C0.ld, rows, cols)
    got = C.window()[rows, cols].astype(np.float64)
    if p.dtype == DTYPE_F32:
        err = float(np.max(np.abs(got - ref)))
        tol = fp32_tol(p, A, B, C0)
        assert err <= tol, f"max |C - C_ref| over samples = {err:.3e} > {tol:.3e}"
        return err
    rel = float(np.linalg.norm(got - ref) / np.linalg.norm(ref))
    assert rel <= 1e-3, f"relative Frobenius error over samples {rel:.3e} > 1e-3"
    return rel
