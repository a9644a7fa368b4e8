"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element, on shapes that
span several tiles with ragged tails, all transpose combinations, padded leading dimensions, and the
degenerate cases.  Tolerances: bit-exact on integer-valued inputs; fp32 max |C - C_ref| <=
4*2^-24*(k*|alpha|*max|A|*max|B| + |beta|*max|C0|); fp16/bf16 relative Frobenius error <= 1e-3 against the
fp64 oracle on the same rounded inputs."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import paper_2310_17408_b200 as g
from workloads import DTYPE_BF16, DTYPE_F16, DTYPE_F32, Problem, make_matrix

from gpu_util import check_against_oracle, drop_workspace, ensure_workspace, run_problem

pytestmark = pytest.mark.gpu

SHAPES = [(1, 1, 1), (64, 64, 64), (129, 257, 65), (200, 300, 150), (5, 1000, 33), (1000, 5, 70),
          (257, 129, 1030), (130, 70, 17), (384, 512, 256)]
TRANS = list(itertools.product("NT", "NT"))
FAMILIES = {DTYPE_F32: [g.GEMM_KERNEL_SIMT_GENERIC, g.GEMM_KERNEL_SIMT_FAST],
            DTYPE_F16: [g.GEMM_KERNEL_SIMT_GENERIC, g.GEMM_KERNEL_TENSOR],
            DTYPE_BF16: [g.GEMM_KERNEL_SIMT_GENERIC, g.GEMM_KERNEL_TENSOR]}


@pytest.fixture(autouse=True)
def _reset_forcing():
    yield
    g.gemm_force_kernel(g.GEMM_KERNEL_AUTO)
    g.gemm_force_tile(0, 0, 0)


def problem(dtype, m, n, k, ta, tb, alpha, beta, kind, pad, seed=1):
    kindA = kindB = kind
    return Problem("t", dtype, m, n, k, alpha, beta, ta, tb, kindA=kindA, kindB=kindB, kindC=kind if kind == "int" else "uniform",
                   seed=seed, pad=pad)


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_F16, DTYPE_BF16])
@pytest.mark.parametrize("ta,tb", TRANS)
def test_parity_grid(dtype, ta, tb):
    kind = "uniform" if dtype == DTYPE_F32 else "normal"
    for family in FAMILIES[dtype]:
        g.gemm_force_kernel(family)
        for (m, n, k) in SHAPES:
            for (alpha, beta), pad in [((1.0, 0.0), (0, 0, 0)), ((1.5, 0.5), (8, 8, 4)), ((-0.75, 1.0), (1, 3, 1))]:
                p = problem(dtype, m, n, k, ta, tb, alpha, beta, kind, pad, seed=m + n + k)
                A, B, C0 = p.operands()
                C, cfg = run_problem(p, A, B, C0)
                check_against_oracle(p, A, B, C0, C)
                if family == g.GEMM_KERNEL_SIMT_GENERIC:
                    assert cfg["kernel"] == g.GEMM_KERNEL_SIMT_GENERIC
                # integer-valued inputs: bit-exact
                p = problem(dtype, m, n, k, ta, tb, alpha, beta, "int", pad, seed=7 + m)
                A, B, C0 = p.operands()
                C, cfg = run_problem(p, A, B, C0)
                check_against_oracle(p, A, B, C0, C, integer=True)


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_F16, DTYPE_BF16])
def test_every_tile_and_split_k(dtype):
    ensure_workspace(256 << 20)
    tiles = [(128, 128), (128, 64), (64, 128), (64, 64)] if dtype == DTYPE_F32 else [(128, 256), (128, 128), (128, 64)]
    kind = "uniform" if dtype == DTYPE_F32 else "normal"
    for (tm, tn), split in itertools.product(tiles, (1, 2, 5)):
        g.gemm_force_tile(tm, tn, split)
        for ta, tb in TRANS:
            p = problem(dtype, 300, 520, 777, ta, tb, 1.5, 0.5, kind, (0, 8, 2), seed=tm + tn + split)
            A, B, C0 = p.operands()
            C, cfg = run_problem(p, A, B, C0)
            assert (cfg["tile_m"], cfg["tile_n"]) == (tm, tn), cfg
            assert cfg["split_k"] == split or (split > 1 and cfg["split_k"] > 1), cfg
            check_against_oracle(p, A, B, C0, C)
            p = problem(dtype, 300, 520, 777, ta, tb, 1.5, 0.5, "int", (0, 8, 2), seed=3)
            A, B, C0 = p.operands()
            C, cfg = run_problem(p, A, B, C0)
            check_against_oracle(p, A, B, C0, C, integer=True)


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_cta_pair_tiles(dtype):
    """256 x 256 tiles on CTA pairs (two SMs per tile): every transpose combination, split-k, tiles whose second
    half lies partly or wholly outside the matrix, and more tiles than pairs (each pair walks several tiles and
    reuses both accumulators and every pipeline stage several times)."""
    ensure_workspace(256 << 20)
    shapes = [(300, 520, 777), (129, 300, 200), (100, 520, 130), (1000, 1100, 264)]
    for split in (1, 2, 3):
        g.gemm_force_tile(256, 256, split)
        for (m, n, k), (ta, tb) in itertools.product(shapes, TRANS):
            p = problem(dtype, m, n, k, ta, tb, 1.5, 0.5, "normal", (8, 0, 4), seed=m + split)
            A, B, C0 = p.operands()
            C, cfg = run_problem(p, A, B, C0)
            assert (cfg["kernel"], cfg["tile_m"], cfg["tile_n"]) == (g.GEMM_KERNEL_TENSOR, 256, 256), cfg
            assert cfg["split_k"] == split or (split > 1 and cfg["split_k"] > 1), cfg
            check_against_oracle(p, A, B, C0, C)
            p = problem(dtype, m, n, k, ta, tb, 1.5, 0.5, "int", (0, 8, 0), seed=5)
            A, B, C0 = p.operands()
            C, cfg = run_problem(p, A, B, C0)
            check_against_oracle(p, A, B, C0, C, integer=True)
    g.gemm_force_tile(256, 256, 1)
    for ta, tb in (("N", "N"), ("T", "N")):
        p = problem(dtype, 2400, 4000, 136, ta, tb, 1.0, 0.0, "int", (0, 0, 0), seed=11)     # 160 tiles
        A, B, C0 = p.operands()
        C, cfg = run_problem(p, A, B, C0)
        assert (cfg["tile_m"], cfg["tile_n"]) == (256, 256) and cfg["grid"] % 2 == 0, cfg
        check_against_oracle(p, A, B, C0, C, integer=True)


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_F16, DTYPE_BF16])
def test_results_are_deterministic(dtype):
    ensure_workspace(64 << 20)
    p = problem(dtype, 256, 256, 4096, "N", "N", 1.0, 0.0, "uniform", (0, 0, 0))
    A, B, C0 = p.operands()
    C1, cfg1 = run_problem(p, A, B, C0)
    C2, cfg2 = run_problem(p, A, B, C0)
    assert cfg1 == cfg2
    assert np.array_equal(C1.buf.view(np.uint32), C2.buf.view(np.uint32))


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_F16])
def test_unaligned_operands_take_a_working_path(dtype):
    # odd leading dimensions and pointers offset by one element: no 16-byte alignment anywhere
    m, n, k = 150, 260, 147
    p = problem(dtype, m, n, k, "N", "N", 1.0, 0.0, "uniform", (1, 0, 1))
    A, B, C0 = p.operands()
    for ws in (True, False):
        if not ws:
            drop_workspace()
        C, cfg = run_problem(p, A, B, C0, workspace=ws)
        check_against_oracle(p, A, B, C0, C)
        if dtype == DTYPE_F16:
            assert (cfg["kernel"] == g.GEMM_KERNEL_TENSOR and cfg["repacked"] == 3) if ws else \
                (cfg["kernel"] == g.GEMM_KERNEL_SIMT_GENERIC)
    # pointers offset by one element
    es = 4 if dtype == DTYPE_F32 else 2
    from gpu_util import to_device
    dA, dB, dC = to_device(A), to_device(B), to_device(C0)
    big = torch.empty(dA.numel() + 1, dtype=dA.dtype, device="cuda")
    big[1:] = dA
    rc = g.gemm(dtype, "N", "N", m, n, k, 1.0, big.data_ptr() + es, A.ld, dB.data_ptr(), B.ld, 0.0, dC.data_ptr(), C0.ld,
                torch.cuda.current_stream().cuda_stream)
    assert rc == 0 and g.gemm_poll_status() == 0
    from workloads import Matrix
    C = Matrix(dC.cpu().numpy(), m, n, C0.ld, DTYPE_F32)
    check_against_oracle(p, A, B, C0, C)


def test_degenerate_cases():
    s = torch.cuda.current_stream().cuda_stream
    C0 = make_matrix(40, 30, kind="uniform", seed=2, matrix_id=2, ld=44)
    A = make_matrix(40, 16, kind="uniform", seed=2, matrix_id=0)
    B = make_matrix(16, 30, kind="uniform", seed=2, matrix_id=1)
    from gpu_util import to_device
    dA, dB = to_device(A), to_device(B)

    def call(m, n, k, alpha, beta, c_init=None, a=dA, b=dB):
        dC = to_device(C0) if c_init is None else c_init.clone()
        rc = g.gemm(DTYPE_F32, "N", "N", m, n, k, alpha, a.data_ptr() if a is not None else 0, 40,
                    b.data_ptr() if b is not None else 0, 16, beta, dC.data_ptr(), 44, s)
        assert rc == 0, g.gemm_status_string(rc)
        assert g.gemm_poll_status() == 0
        return dC.cpu().numpy()

    base = C0.buf
    # m == 0 or n == 0: nothing happens
    assert np.array_equal(call(0, 30, 16, 1.0, 0.0).view(np.uint32), base.view(np.uint32))
    assert np.array_equal(call(40, 0, 16, 1.0, 0.0).view(np.uint32), base.view(np.uint32))
    # k == 0 / alpha == 0: C <- beta*C, A and B may be null
    want = C0.copy(); want.window()[:] = 0.5 * C0.window()
    assert np.array_equal(call(40, 30, 0, 1.0, 0.5, a=None, b=None).view(np.uint32), want.buf.view(np.uint32))
    assert np.array_equal(call(40, 30, 16, 0.0, 0.5, a=None, b=None).view(np.uint32), want.buf.view(np.uint32))
    # beta == 1 with nothing to add: untouched
    assert np.array_equal(call(40, 30, 16, 0.0, 1.0).view(np.uint32), base.view(np.uint32))
    # beta == 0: C is write-only, NaN/Inf in it must not propagate (also through the main kernels)
    nanC = torch.full((44 * 30,), float("nan"), device="cuda")
    out = call(40, 30, 0, 1.0, 0.0, c_init=nanC).reshape(30, 44)
    assert np.all(out[:, :40] == 0.0) and np.all(np.isnan(out[:, 40:]))
    out = call(40, 30, 16, 1.0, 0.0, c_init=nanC).reshape(30, 44)
    assert np.all(np.isfinite(out[:, :40])) and np.all(np.isnan(out[:, 40:]))
    ref = A.as_f64() @ B.as_f64()
    assert np.max(np.abs(out[:, :40].T - ref)) < 1e-5
    for dt in (DTYPE_F16, DTYPE_BF16):
        Ah = make_matrix(40, 16, kind="int", seed=2, matrix_id=0, dtype=dt)
        Bh = make_matrix(16, 30, kind="int", seed=2, matrix_id=1, dtype=dt)
        dAh, dBh = to_device(Ah), to_device(Bh)
        dC = nanC.clone()
        assert g.gemm(dt, "N", "N", 40, 30, 16, 1.0, dAh.data_ptr(), 40, dBh.data_ptr(), 16, 0.0, dC.data_ptr(), 44, s) == 0
        out = dC.cpu().numpy().reshape(30, 44)
        assert np.array_equal(out[:, :40].T, Ah.as_f64() @ Bh.as_f64())


def test_invalid_arguments_launch_nothing():
    C = torch.full((64,), 7.0, device="cuda")
    A = torch.zeros(64, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    a, c = A.data_ptr(), C.data_ptr()
    cases = [((9, "N", "N", 8, 8, 8, 1.0, a, 8, a, 8, 0.0, c, 8), -1),
             ((0, "X", "N", 8, 8, 8, 1.0, a, 8, a, 8, 0.0, c, 8), -2),
             ((0, "N", "Q", 8, 8, 8, 1.0, a, 8, a, 8, 0.0, c, 8), -3),
             ((0, "N", "N", -1, 8, 8, 1.0, a, 8, a, 8, 0.0, c, 8), -4),
             ((0, "N", "N", 8, -1, 8, 1.0, a, 8, a, 8, 0.0, c, 8), -5),
             ((0, "N", "N", 8, 8, -1, 1.0, a, 8, a, 8, 0.0, c, 8), -6),
             ((0, "N", "N", 8, 8, 8, 1.0, 0, 8, a, 8, 0.0, c, 8), -8),
             ((0, "N", "N", 8, 8, 8, 1.0, a, 7, a, 8, 0.0, c, 8), -9),
             ((0, "T", "N", 8, 8, 4, 1.0, a, 3, a, 8, 0.0, c, 8), -9),
             ((0, "N", "N", 8, 8, 8, 1.0, a, 8, 0, 8, 0.0, c, 8), -10),
             ((0, "N", "N", 8, 8, 8, 1.0, a, 8, a, 7, 0.0, c, 8), -11),
             ((0, "N", "N", 8, 8, 8, 1.0, a, 8, a, 8, 0.0, 0, 8), -13),
             ((0, "N", "N", 8, 8, 8, 1.0, a, 8, a, 8, 0.0, c, 7), -14)]
    for args, want in cases:
        assert g.gemm(*args, s) == want, (args, want)
        assert g.gemm_status_string(want).startswith("invalid argument")
    torch.cuda.synchronize()
    assert torch.all(C == 7.0)


def test_bounded_wait_expiry_is_reported_and_context_survives():
    # a wait that can never be satisfied gives up after its limit: status word set, kernel exits, nothing faults
    s = torch.cuda.current_stream().cuda_stream
    assert g.gemm_poll_status() == 0
    assert g.gemm_selftest_wait_expiry(s) == 0
    assert g.gemm_poll_status() == g.GEMM_ERR_DEVICE
    detail = g.gemm_status_detail()
    assert detail >> 24 == 0xE5 and (detail >> 16) & 0xFF == 0x7F, hex(detail)
    assert g.gemm_status_string(g.GEMM_ERR_DEVICE) == "a bounded device-side wait expired"
    assert g.gemm_poll_status() == 0                      # cleared by the poll
    # the context is still usable: a tensor-core GEMM right after it is correct
    p = problem(DTYPE_BF16, 200, 300, 150, "N", "N", 1.0, 0.0, "int", (0, 0, 0))
    A, B, C0 = p.operands()
    C, cfg = run_problem(p, A, B, C0)
    check_against_oracle(p, A, B, C0, C, integer=True)


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_BF16])
def test_gemm_host_pipelined_panels_match_oracle(dtype):
    # host-buffer entry point: several column panels in flight (large n), padded leading dimensions, both B layouts
    kind = "uniform" if dtype == DTYPE_F32 else "normal"
    cases = [(300, 9000, 700, "N", "N", 1.5, 0.5, (4, 8, 4)),      # multi-panel, C read and written
             (260, 8200, 1100, "T", "T", 1.0, 0.0, (8, 8, 2)),     # multi-panel, strided panels of B, C write-only
             (100, 90, 70, "N", "T", -1.0, 1.0, (1, 3, 1)),        # single panel
             (4500, 3000, 2100, "N", "N", 1.0, 0.5, (4, 0, 4)),    # A large enough to arrive in row panels
             (4400, 2900, 2050, "T", "N", 1.0, 0.0, (8, 8, 0)),    # same with A stored transposed
             (4300, 2800, 2200, "N", "T", 1.5, 0.5, (0, 8, 4)),    # k slices of a transposed B beside A's
             (40, 50, 0, "N", "N", 1.0, 0.5, (0, 0, 2)),           # k = 0: only beta*C
             (300, 2000, 0, "T", "N", 1.0, 0.0, (0, 0, 0)),        # k = 0, several panels, C overwritten with zeros
             (64, 1500, 33, "N", "N", 0.0, -2.0, (1, 1, 1))]       # alpha = 0: A and B are not read
    for (m, n, k, ta, tb, alpha, beta, pad) in cases:
        p = problem(dtype, m, n, k, ta, tb, alpha, beta, kind, pad, seed=m)
        A, B, C0 = p.operands()
        C = C0.copy()
        if beta == 0.0:
            C.window()[:] = np.nan                                  # must be overwritten, never read
        rc = g.gemm_host(dtype, ta, tb, m, n, k, alpha, A.buf.ctypes.data, A.ld, B.buf.ctypes.data, B.ld, beta,
                         C.buf.ctypes.data, C.ld, torch.cuda.current_stream().cuda_stream)
        assert rc == 0, g.gemm_status_string(rc)
        assert C.padding_intact()
        check_against_oracle(p, A, B, C0, C)


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_BF16])
def test_concurrent_host_threads_on_their_own_streams(dtype):
    # calls from different host threads on different streams are independent when no workspace is registered
    import threading
    drop_workspace()
    kind = "uniform" if dtype == DTYPE_F32 else "normal"
    results, errors = {}, []

    def worker(idx):
        try:
            torch.cuda.set_device(0)
            stream = torch.cuda.Stream()
            p = problem(dtype, 260 + 64 * idx, 390, 700 + 100 * idx, "N", "T" if idx % 2 else "N", 1.5, 0.5, kind, (0, 0, 0),
                        seed=50 + idx)
            A, B, C0 = p.operands()
            from gpu_util import to_device
            with torch.cuda.stream(stream):
                dA, dB, dC = to_device(A), to_device(B), to_device(C0)
                for _ in range(20):                      # keep both streams busy at the same time
                    dC.copy_(torch.from_numpy(C0.buf), non_blocking=False)
                    rc = g.gemm(dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, dA.data_ptr(), A.ld, dB.data_ptr(),
                                B.ld, p.beta, dC.data_ptr(), C0.ld, stream.cuda_stream)
                    assert rc == 0
                stream.synchronize()
                from workloads import Matrix
                results[idx] = (p, A, B, C0, Matrix(dC.cpu().numpy(), p.m, p.n, C0.ld, DTYPE_F32))
        except Exception as exc:      # surfaced in the main thread
            errors.append(exc)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(3)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert g.gemm_poll_status() == 0
    for idx, (p, A, B, C0, C) in results.items():
        check_against_oracle(p, A, B, C0, C)


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_F16, DTYPE_BF16])
def test_nan_and_inf_in_operands_stay_in_their_rows_and_columns(dtype):
    # a NaN in row 5 of A poisons row 5 of C, an Inf in column 7 of B makes column 7 of C non-finite; nothing else changes
    from gpu_util import to_device
    from workloads import Matrix, encode_bf16, encode_f16
    m, n, k = 200, 300, 130
    p = problem(dtype, m, n, k, "N", "N", 1.0, 0.0, "int", (0, 0, 0), seed=4)
    A, B, C0 = p.operands()
    clean, _ = run_problem(p, A, B, C0)
    A2, B2 = A.copy(), B.copy()
    nan = {DTYPE_F32: np.float32("nan"), DTYPE_F16: encode_f16(np.array([np.nan]))[0], DTYPE_BF16: encode_bf16(np.array([np.nan]))[0]}[dtype]
    inf = {DTYPE_F32: np.float32("inf"), DTYPE_F16: encode_f16(np.array([np.inf]))[0], DTYPE_BF16: encode_bf16(np.array([np.inf]))[0]}[dtype]
    A2.window()[5, 17] = nan
    B2.window()[40, 7] = inf
    dirty, _ = run_problem(p, A2, B2, C0)
    d, c = dirty.window(), clean.window()
    assert np.all(np.isnan(d[5, :]))
    assert not np.any(np.isfinite(d[:, 7]))
    mask = np.ones((m, n), dtype=bool)
    mask[5, :] = False
    mask[:, 7] = False
    assert np.array_equal(d[mask], c[mask])


def test_fp16_subnormal_inputs_are_not_flushed():
    # binary16 subnormals (multiples of 2^-24 below 2^-14) times small integers: every product and sum is exact in
    # fp32, so the tensor-core result must equal the fp64 oracle exactly if subnormal inputs are honoured
    from workloads import Matrix, encode_f16
    m, n, k = 128, 128, 64
    rng = np.random.default_rng(3)
    a = rng.integers(1, 1000, (m, k)).astype(np.float64) * 2.0 ** -24          # all subnormal in binary16
    b = rng.integers(-4, 5, (k, n)).astype(np.float64)
    A = Matrix(encode_f16(a.T.ravel()).copy(), m, k, m, DTYPE_F16)              # column-major buffers
    B = Matrix(encode_f16(b.T.ravel()).copy(), k, n, k, DTYPE_F16)
    assert np.array_equal(A.as_f64(), a) and np.all(np.abs(a) < 2.0 ** -14)
    C0 = make_matrix(m, n, kind="zeros", seed=0, matrix_id=2)
    p = Problem("sub", DTYPE_F16, m, n, k, 1.0, 0.0)
    C, cfg = run_problem(p, A, B, C0)
    assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR
    assert np.array_equal(C.window().astype(np.float64), a @ b)


def test_fp32_tail_split_of_the_last_wave():
    # more tiles than CTA slots with a small remainder: the tiles of the last wave are cut along k and finished by
    # the tail reduction; ragged edges, all transpose combinations, integer-exact and random data
    ensure_workspace(64 << 20)
    for ta, tb in TRANS:
        for (m, n, k) in [(2048, 2560, 2100), (2000, 2590, 1030), (4100, 1300, 777)]:
            p = problem(DTYPE_F32, m, n, k, ta, tb, 1.5, 0.5, "uniform", (0, 4, 0), seed=m)
            A, B, C0 = p.operands()
            C, cfg = run_problem(p, A, B, C0)
            assert cfg["tail_split"] >= 2 and cfg["split_k"] == 1 and cfg["launches"] == 2, cfg
            check_against_oracle(p, A, B, C0, C)
        p = problem(DTYPE_F32, 2000, 2590, 1030, ta, tb, -1.0, 1.0, "int", (4, 0, 4), seed=9)
        A, B, C0 = p.operands()
        C, cfg = run_problem(p, A, B, C0)
        assert cfg["tail_split"] >= 2
        check_against_oracle(p, A, B, C0, C, integer=True)
    # without a workspace the same problem runs unsplit
    drop_workspace()
    p = problem(DTYPE_F32, 2048, 2560, 2100, "N", "N", 1.0, 0.0, "uniform", (0, 0, 0), seed=1)
    A, B, C0 = p.operands()
    C, cfg = run_problem(p, A, B, C0, workspace=False)
    assert cfg["tail_split"] == 0
    check_against_oracle(p, A, B, C0, C)


@pytest.mark.parametrize("api_dtype", [DTYPE_F16, DTYPE_BF16, g.GEMM_F16_C16, g.GEMM_BF16_C16, DTYPE_F32])
def test_nothing_is_written_outside_the_m_by_n_window(api_dtype):
    """C sits in the middle of a larger buffer filled with a sentinel: the elements before it, the rows m..ldc-1 of
    every column and everything after column n-1 must keep it.  The shapes end inside a tile in both directions and
    take the TMA tile stores (columns ending on 16-byte boundaries) as well as the direct stores."""
    s = torch.cuda.current_stream().cuda_stream
    in_t = {DTYPE_F32: torch.float32, DTYPE_F16: torch.float16, DTYPE_BF16: torch.bfloat16,
            g.GEMM_F16_C16: torch.float16, g.GEMM_BF16_C16: torch.bfloat16}[api_dtype]
    out_t = in_t if api_dtype in (g.GEMM_F16_C16, g.GEMM_BF16_C16) else torch.float32
    ensure_workspace(64 << 20)
    for (m, n, k, ldc) in [(136, 257, 64, 136), (136, 257, 64, 144), (130, 300, 64, 136), (264, 70, 48, 272), (8, 1000, 40, 16)]:      # |sums| <= 256: exact in bf16 too
        A = torch.randint(-2, 3, (k * m,), device="cuda").to(in_t)
        B = torch.randint(-2, 3, (n * k,), device="cuda").to(in_t)
        guard = 4096
        buf = torch.full((guard + ldc * n + guard,), 7.0, device="cuda", dtype=out_t)
        C = buf[guard:]
        rc = g.gemm(api_dtype, "N", "N", m, n, k, 1.0, A.data_ptr(), m, B.data_ptr(), k, 0.0, C.data_ptr(), ldc, s)
        assert rc == 0 and g.gemm_poll_status() == 0
        host = buf.float().cpu().numpy()
        body = host[guard:guard + ldc * n].reshape(n, ldc)
        # expected values from the CPU oracle's definition layer (small integers: exact in every type involved)
        in_code = {DTYPE_F32: DTYPE_F32, DTYPE_F16: DTYPE_F16, DTYPE_BF16: DTYPE_BF16,
                   g.GEMM_F16_C16: DTYPE_F16, g.GEMM_BF16_C16: DTYPE_BF16}[api_dtype]
        bits = (lambda t: t.cpu().numpy()) if in_code == DTYPE_F32 else (lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16))
        want = oracle.gemm_l0(in_code, "N", "N", m, n, k, 1.0, bits(A), m, bits(B), k, 0.0,
                              np.zeros(m * n, dtype=np.float32), m, acc=oracle.ACC_F32)
        assert np.array_equal(body[:, :m], want.T), (m, n, k, ldc)
        assert np.all(body[:, m:] == 7.0), "rows m..ldc-1 were written"
        assert np.all(host[:guard] == 7.0) and np.all(host[guard + ldc * n:] == 7.0), "written outside the buffer of C"


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
@pytest.mark.parametrize("ta,tb", TRANS)
def test_few_rows_many_columns_take_the_exchanged_operand_roles(dtype, ta, tb):
    """16-bit inputs, at most 64 rows of C, many columns (the C_out = 64 layers): the library computes C^T = op(B)^T op(A)^T
    with the columns of C as the rows of the MMA.  Ragged sizes, padded and unaligned leading dimensions (C then takes
    the scalar stores, the operands the aligned copy), alpha / beta, exact integers."""
    ensure_workspace(64 << 20)
    for (m, n, k), pad in [((64, 2048, 128), (0, 0, 0)), ((64, 1500, 200), (0, 0, 0)), ((17, 4100, 70), (8, 8, 4)),
                           ((1, 1024, 64), (0, 0, 3)), ((40, 1100, 147), (1, 1, 1))]:
        for kind, alpha, beta in [("int", 1.5, 0.5), ("normal", 1.0, 0.0), ("normal", -0.75, 1.25)]:
            p = problem(dtype, m, n, k, ta, tb, alpha, beta, kind, pad, seed=n + k)
            A, B, C0 = p.operands()
            C, cfg = run_problem(p, A, B, C0)
            assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR and (cfg["tile_m"], cfg["tile_n"]) == (64, 128), cfg
            check_against_oracle(p, A, B, C0, C, integer=(kind == "int"))
    # a forced tile keeps the operands' roles: same result within the tolerance, the other kernel
    p = problem(dtype, 64, 2048, 256, ta, tb, 1.0, 0.0, "int", (0, 0, 0), seed=5)
    A, B, C0 = p.operands()
    C1, cfg1 = run_problem(p, A, B, C0)
    g.gemm_force_tile(128, 256, 0)
    C2, cfg2 = run_problem(p, A, B, C0)
    assert (cfg1["tile_m"], cfg1["tile_n"]) == (64, 128) and (cfg2["tile_m"], cfg2["tile_n"]) == (128, 256)
    assert np.array_equal(C1.buf.view(np.uint32), C2.buf.view(np.uint32))
