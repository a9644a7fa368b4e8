"""gemm_strided_batched and the small-problem kernels against the CPU oracle (one gemm_l0 / gemm_l1 call per problem of
the batch): integer-valued data bit for bit, random data within the fp32 bound (16-bit inputs: relative Frobenius
error), over transpose flags, ragged sizes, padded leading dimensions, shared operands (stride 0), batch = 1 and
batches beyond one launch's grid limit; the kernel without operand staging also through gemm() itself; and the two
ways of finishing a split of k (separate pass over the workspace, thread-block cluster inside the kernel) against each other."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import paper_2310_17408_b200 as g
from workloads import DTYPE_BF16, DTYPE_F16, DTYPE_F32, Problem, make_matrix

from gpu_util import check_against_oracle, ensure_workspace, run_problem, to_device

pytestmark = pytest.mark.gpu
TRANS = list(itertools.product("NT", "NT"))


@pytest.fixture(autouse=True)
def _reset_forcing():
    yield
    g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
    g.gemm_force_tile(0, 0, 0)
    g.gemm_force_reduction(0)


def make_batch(dtype, m, n, k, ta, tb, batch, kind, seed, pad=(0, 0, 0), gap=(0, 0, 0), shared_a=False, shared_b=False):
    """Host operands of a strided batch: per problem one stored A, B, C0 (column-major, padded leading dimensions),
    laid out `stride` elements apart (stride = ld*cols + gap).  Returns the flat buffers, strides and per-problem matrices."""
    (ar, ac), (br, bc) = ((m, k) if ta == "N" else (k, m)), ((k, n) if tb == "N" else (n, k))
    kindc = kind if kind == "int" else "uniform"
    mats = []
    for b in range(batch):
        A = make_matrix(ar, ac, kind=kind, seed=seed + (0 if shared_a else b), matrix_id=0, dtype=dtype, ld=max(1, ar) + pad[0])
        B = make_matrix(br, bc, kind=kind, seed=seed + (0 if shared_b else b), matrix_id=1, dtype=dtype, ld=max(1, br) + pad[1])
        C = make_matrix(m, n, kind=kindc, seed=seed + b, matrix_id=2, ld=max(1, m) + pad[2])
        mats.append((A, B, C))
    A0, B0, C0 = mats[0]
    sA = 0 if shared_a else A0.buf.size + gap[0]
    sB = 0 if shared_b else B0.buf.size + gap[1]
    sC = C0.buf.size + gap[2]

    def flat(idx, stride, shared):
        first = mats[0][idx].buf
        if shared:
            return first.copy()
        out = np.zeros(stride * batch, dtype=first.dtype)
        for b in range(batch):
            out[b * stride: b * stride + first.size] = mats[b][idx].buf
        return out
    return flat(0, sA, shared_a), flat(1, sB, shared_b), flat(2, sC, False), (sA, sB, sC), mats


def run_batched(dtype, m, n, k, ta, tb, alpha, beta, batch, kind, seed=7, **kw):
    hA, hB, hC, (sA, sB, sC), mats = make_batch(dtype, m, n, k, ta, tb, batch, kind, seed, **kw)
    dev = lambda x: torch.from_numpy(x.view(np.int16) if x.dtype == np.uint16 else x).cuda()
    dA, dB, dC = dev(hA), dev(hB), dev(hC)
    A0, B0, C0 = mats[0]
    rc = g.gemm_strided_batched(dtype, ta, tb, m, n, k, alpha, dA.data_ptr(), A0.ld, sA, dB.data_ptr(), B0.ld, sB, beta,
                                dC.data_ptr(), C0.ld, sC, batch, torch.cuda.current_stream().cuda_stream)
    assert rc == 0, rc
    cfg = g.gemm_last_config()
    assert g.gemm_poll_status() == 0, hex(g.gemm_status_detail())
    out = dC.cpu().numpy()
    worst = 0.0
    for b, (A, B, C) in enumerate(mats):
        got_full = out[b * sC: b * sC + C.buf.size].reshape(n, C.ld)
        got = got_full[:, :m].T
        # padding rows of every problem keep their canaries; the gap between problems keeps its zeros
        assert np.array_equal(got_full[:, m:].view(np.uint32), C.buf.reshape(n, C.ld)[:, m:].view(np.uint32))
        args = (dtype, ta, tb, m, n, k, alpha, A.buf, A.ld, B.buf, B.ld, beta, C.buf, C.ld)
        if kind == "int":
            want = oracle.gemm_l0(*args, acc=oracle.ACC_F32)
            assert np.array_equal(np.ascontiguousarray(got).view(np.uint32), np.ascontiguousarray(want).view(np.uint32)), (b, cfg)
        else:
            ref = oracle.gemm_l0(*args, acc=oracle.ACC_F64)
            if dtype == DTYPE_F32:
                tol = oracle.fp32_tolerance(k, alpha, beta, A.max_abs(), B.max_abs(), C.max_abs() if beta else 0.0)
                err = float(np.max(np.abs(got.astype(np.float64) - ref))) if ref.size else 0.0
                assert err <= tol, (b, err, tol, cfg)
                worst = max(worst, err)
            else:
                den = np.linalg.norm(ref)
                rel = float(np.linalg.norm(got.astype(np.float64) - ref) / den) if den else 0.0
                assert rel <= 1e-3, (b, rel, cfg)
        gap_part = out[b * sC + C.buf.size: (b + 1) * sC]
        assert not gap_part.size or np.all(gap_part == 0)
    return cfg


SHAPES = [(1, 1, 1), (5, 7, 3), (16, 16, 16), (33, 65, 17), (64, 64, 64), (96, 96, 200), (130, 70, 40)]


@pytest.mark.parametrize("ta,tb", TRANS)
@pytest.mark.parametrize("force", [g.GEMM_KERNEL_AUTO, g.GEMM_KERNEL_SIMT_DIRECT, g.GEMM_KERNEL_SIMT_FAST, g.GEMM_KERNEL_SIMT_GENERIC])
def test_batched_fp32_grid(ta, tb, force):
    for (m, n, k) in SHAPES:
        for batch, kind, alpha, beta, pad, gap in [(1, "int", 1.5, 0.5, (0, 0, 0), (0, 0, 0)), (3, "int", -1.0, 1.0, (1, 2, 3), (5, 0, 7)),
                                                     (7, "uniform", 1.25, 0.0, (4, 4, 4), (0, 4, 8)), (4, "uniform", 0.75, -0.5, (0, 0, 0), (0, 0, 0))]:
            g.gemm_force_kernel(force)
            cfg = run_batched(DTYPE_F32, m, n, k, ta, tb, alpha, beta, batch, kind, seed=11 + m, pad=pad, gap=gap)
            if force != g.GEMM_KERNEL_AUTO:
                assert cfg["kernel"] == force, cfg
            assert cfg["launches"] == 1


def test_batched_shared_operands_and_scaling_only():
    # stride 0: every problem multiplies by the same A (or the same B)
    run_batched(DTYPE_F32, 48, 40, 72, "N", "N", 1.0, 0.0, 5, "int", shared_a=True)
    run_batched(DTYPE_F32, 48, 40, 72, "T", "T", 1.5, 0.5, 5, "uniform", shared_b=True)
    # alpha = 0: C <- beta*C for every problem, operands not read; k = 0 likewise
    cfg = run_batched(DTYPE_F32, 20, 30, 16, "N", "N", 0.0, 0.5, 6, "int", pad=(0, 0, 2), gap=(0, 0, 3))
    assert cfg["kernel"] == g.GEMM_KERNEL_SCALE_ONLY
    run_batched(DTYPE_F32, 20, 30, 0, "N", "N", 1.0, 0.0, 3, "int")


def test_batched_beyond_one_launch():
    # more problems than the batch dimension of a grid holds (65535).  All problems share A and B (stride 0) and start
    # from their own C, so one oracle call per distinct C0 value gives every expected result.  The kernel without
    # staging numbers its work units through the whole batch (one launch); the staged kernel runs in two launches.
    m, n, k, batch = 4, 4, 8, 70000
    A = make_matrix(m, k, kind="int", seed=1, matrix_id=0)
    B = make_matrix(k, n, kind="int", seed=1, matrix_id=1)
    c0 = (np.arange(batch, dtype=np.float32) % 5.0) - 2.0                  # problem b starts from the constant (b mod 5) - 2
    hC = np.repeat(c0, m * n).astype(np.float32)
    dA, dB = to_device(A), to_device(B)
    for force, launches in ((g.GEMM_KERNEL_AUTO, 1), (g.GEMM_KERNEL_SIMT_FAST, 2)):
        dC = torch.from_numpy(hC).cuda()
        g.gemm_force_kernel(force)
        rc = g.gemm_strided_batched(DTYPE_F32, "N", "N", m, n, k, 1.0, dA.data_ptr(), m, 0, dB.data_ptr(), k, 0, 0.5,
                                    dC.data_ptr(), m, m * n, batch, torch.cuda.current_stream().cuda_stream)
        assert rc == 0
        cfg = g.gemm_last_config()
        assert cfg["launches"] == launches, cfg
        assert cfg["kernel"] == (g.GEMM_KERNEL_SIMT_DIRECT if force == g.GEMM_KERNEL_AUTO else g.GEMM_KERNEL_SIMT_FAST)
        assert g.gemm_poll_status() == 0
        got = dC.cpu().numpy().reshape(batch, n, m)
        for v in range(5):
            C0 = np.full(m * n, v - 2.0, dtype=np.float32)
            want = oracle.gemm_l0(DTYPE_F32, "N", "N", m, n, k, 1.0, A.buf, m, B.buf, k, 0.5, C0, m, acc=oracle.ACC_F32)
            assert np.array_equal(got[v::5], np.broadcast_to(want.T, got[v::5].shape))


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_batched_16bit_inputs(dtype):
    for ta, tb in TRANS:
        cfg = run_batched(dtype, 40, 56, 72, ta, tb, 1.5, 0.5, 5, "int", pad=(8, 0, 1))
        assert cfg["kernel"] == g.GEMM_KERNEL_SIMT_GENERIC and cfg["launches"] == 1
        run_batched(dtype, 40, 56, 72, ta, tb, 1.0, 0.0, 3, "normal", seed=3)
    # operands TMA cannot address (leading dimension not a multiple of 8): problems large enough for the tensor cores
    # run through gemm() one by one
    ensure_workspace(64 << 20)
    cfg = run_batched(dtype, 256, 264, 320, "N", "N", 1.0, 0.0, 3, "int", pad=(3, 0, 0))
    assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["launches"] >= 3


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
@pytest.mark.parametrize("ta,tb", TRANS)
def test_batched_16bit_on_the_tensor_cores_in_one_launch(dtype, ta, tb):
    # addressable operands (16-byte aligned bases, leading dimensions and batch strides): the whole batch is one launch
    # of the tensor kernel, the problem index being the third coordinate of the operand maps.  Ragged m, n, k (the
    # boxes are clipped per problem), padded leading dimensions, gaps between the problems, C read and written.
    for (m, n, k), batch, pad, gap in [((64, 64, 64), 40, (0, 0, 0), (0, 0, 0)), ((200, 136, 72), 7, (8, 8, 3), (8, 16, 5)),
                                       ((130, 300, 200), 5, (16, 0, 1), (0, 8, 0)), ((8, 520, 1000), 40, (0, 8, 0), (8, 0, 3))]:
        # leading dimensions must come out as multiples of 8: stored rows are m, k or n depending on the flags
        rows_a, rows_b = (m if ta == "N" else k), (k if tb == "N" else n)
        pad_ok = ((-rows_a) % 8 + pad[0], (-rows_b) % 8 + pad[1], pad[2])
        for kind, alpha, beta in (("int", 1.5, 0.5), ("normal", 1.0, 0.0), ("normal", -1.0, 1.0)):
            cfg = run_batched(dtype, m, n, k, ta, tb, alpha, beta, batch, kind, seed=11, pad=pad_ok, gap=gap)
            assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["launches"] == 1, (m, n, k, cfg)


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_batched_16bit_shared_operands_on_the_tensor_cores(dtype):
    for shared in (dict(shared_a=True), dict(shared_b=True), dict(shared_a=True, shared_b=True)):
        cfg = run_batched(dtype, 136, 200, 264, "N", "T", 1.5, 0.5, 6, "int", seed=5, **shared)
        assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["launches"] == 1, cfg
        run_batched(dtype, 136, 200, 264, "T", "N", 1.0, 0.0, 6, "normal", seed=6, **shared)


def test_batched_argument_checks():
    x = torch.zeros(4096, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    p = x.data_ptr()
    ok = dict(dtype=0, ta="N", tb="N", m=8, n=8, k=8, alpha=1.0, A=p, lda=8, sA=64, B=p, ldb=8, sB=64, beta=0.0, C=p, ldc=8, sC=64, batch=2)

    def call(**over):
        a = dict(ok, **over)
        return g.gemm_strided_batched(a["dtype"], a["ta"], a["tb"], a["m"], a["n"], a["k"], a["alpha"], a["A"], a["lda"], a["sA"],
                                      a["B"], a["ldb"], a["sB"], a["beta"], a["C"], a["ldc"], a["sC"], a["batch"], s)
    assert call(dtype=9) == -1 and call(ta="X") == -2 and call(m=-1) == -4 and call(A=0) == -8 and call(lda=7) == -9
    assert call(sA=-1) == -10 and call(B=0) == -11 and call(ldb=7) == -12 and call(sB=-1) == -13 and call(C=0) == -15
    assert call(ldc=7) == -16 and call(sC=63) == -17 and call(batch=-1) == -18
    assert call(batch=0) == 0 and call(m=0) == 0
    torch.cuda.synchronize()
    assert torch.all(x == 0)


@pytest.mark.parametrize("ta,tb", TRANS)
def test_direct_kernel_through_gemm(ta, tb):
    # the selector takes the kernel without staging for tiny fp32 problems; misaligned leading dimensions take its scalar loads
    for (m, n, k), pad in [((64, 64, 64), (0, 0, 0)), ((17, 90, 33), (1, 2, 3)), ((60, 40, 50), (4, 0, 4)), ((1, 1, 5), (0, 0, 0))]:
        for kind, alpha, beta in [("int", 1.5, 0.5), ("uniform", -1.25, 0.0)]:
            p = Problem("tiny", DTYPE_F32, m, n, k, alpha, beta, ta, tb, kindA=kind, kindB=kind, kindC=kind if kind == "int" else "uniform",
                        seed=m + k, pad=pad)
            A, B, C0 = p.operands()
            C, cfg = run_problem(p, A, B, C0)
            assert cfg["kernel"] == g.GEMM_KERNEL_SIMT_DIRECT and cfg["launches"] == 1, cfg
            check_against_oracle(p, A, B, C0, C, integer=(kind == "int"))


@pytest.mark.parametrize("shape", [(512, 512, 512), (256, 256, 4096), (200, 136, 4100), (1024, 64, 2048)])
def test_split_k_finished_in_kernel_equals_the_separate_pass(shape):
    m, n, k = shape
    ensure_workspace(128 << 20)
    for ta, tb in (("N", "N"), ("T", "N"), ("N", "T")):
        p = Problem("sk", DTYPE_F32, m, n, k, 1.5, 0.5, ta, tb, seed=m + k, pad=(0, 0, 0 if m % 4 == 0 else 3))
        A, B, C0 = p.operands()
        g.gemm_force_reduction(2)
        C_in, cfg_in = run_problem(p, A, B, C0)
        assert cfg_in["split_k"] > 1 and cfg_in["launches"] == 1, cfg_in
        check_against_oracle(p, A, B, C0, C_in)
        g.gemm_force_reduction(1)
        g.gemm_force_tile(cfg_in["tile_m"], cfg_in["tile_n"], cfg_in["split_k"])
        C_sep, cfg_sep = run_problem(p, A, B, C0)
        g.gemm_force_tile(0, 0, 0)
        assert cfg_sep["split_k"] == cfg_in["split_k"] and cfg_sep["launches"] == 2, cfg_sep
        # both sum a tile's partial sums in increasing split index and apply the same epilogue: identical bits
        assert np.array_equal(C_in.buf.view(np.uint32), C_sep.buf.view(np.uint32))
        # and again, now without any workspace: the cluster needs none
        from gpu_util import drop_workspace
        drop_workspace()
        g.gemm_force_reduction(0)
        C_again, cfg_again = run_problem(p, A, B, C0, workspace=False)
        assert cfg_again["split_k"] > 1 and cfg_again["launches"] == 1, cfg_again
        if cfg_again["split_k"] == cfg_in["split_k"] and cfg_again["tile_m"] == cfg_in["tile_m"] and cfg_again["tile_n"] == cfg_in["tile_n"]:
            assert np.array_equal(C_in.buf.view(np.uint32), C_again.buf.view(np.uint32))
        check_against_oracle(p, A, B, C0, C_again)
        ensure_workspace(128 << 20)
    # integer data bit for bit against the oracle
    p = Problem("ski", DTYPE_F32, m, n, k, -1.0, 1.0, kindA="int", kindB="int", kindC="int", seed=5)
    A, B, C0 = p.operands()
    g.gemm_force_reduction(2)
    C, cfg = run_problem(p, A, B, C0)
    assert cfg["launches"] == 1
    check_against_oracle(p, A, B, C0, C, integer=True)
