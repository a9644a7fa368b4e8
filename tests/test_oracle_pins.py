"""Pins for the CPU oracle: everything here is fixed by the mathematics or by the paper, not by
the oracle itself (hand-worked products, closed forms, exact integer cases, a library matmul on
special cases, format definitions), so that a dropped term, a wrong sign or index, or a
transposed operand in the oracle fails at least one test."""
import itertools
import os

import numpy as np
import pytest

import oracle
from oracle import ACC_F32, ACC_F32FMA, ACC_F64, OR_BF16, OR_F16, OR_F32
from workloads import (DTYPE_BF16, DTYPE_F16, DTYPE_F32, RESNET50_V15_BATCH1, VGG16_BATCH1,
                       encode_bf16, encode_f16, im2row_shapes, make_matrix)
from workloads.generators import Matrix, decode_16, encode_f16

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def colmajor(a, ld=None, dtype=np.float32):
    """numpy 2-D -> (1-D column-major buffer, ld) with NaN in the padding rows."""
    a = np.asarray(a, dtype=np.float64)
    r, c = a.shape
    ld = max(1, r) if ld is None else ld
    buf = np.full(ld * c, np.nan, dtype=dtype)
    buf.reshape(c, ld).T[:r, :] = a.astype(dtype)
    return buf, ld


def l0(A, B, ta="N", tb="N", alpha=1.0, beta=0.0, C0=None, acc=ACC_F64, lda=None, ldb=None):
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    m = A.shape[0] if ta == "N" else A.shape[1]
    k = A.shape[1] if ta == "N" else A.shape[0]
    n = B.shape[1] if tb == "N" else B.shape[0]
    a, lda = colmajor(A, lda)
    b, ldb = colmajor(B, ldb)
    if C0 is None:
        c0, ldc0 = np.full(max(1, m) * n, np.nan, dtype=np.float32), max(1, m)
    else:
        c0, ldc0 = colmajor(C0)
    return oracle.gemm_l0(OR_F32, ta, tb, m, n, k, alpha, a, lda, b, ldb, beta, c0, ldc0, acc=acc)


# ---------------------------------------------------------------- number formats

def test_decode_f16_all_patterns_against_format_definition():
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    got = np.array([oracle.decode_f16(int(b)) for b in bits])
    both_nan = np.isnan(want) & np.isnan(got)
    assert np.all((want == got) | both_nan)
    assert np.all(np.signbit(want) == np.signbit(got))
    # values fixed by IEEE 754 binary16
    assert oracle.decode_f16(0x3C00) == 1.0
    assert oracle.decode_f16(0xC000) == -2.0
    assert oracle.decode_f16(0x0001) == 2.0 ** -24
    assert oracle.decode_f16(0x7BFF) == 65504.0
    assert oracle.decode_f16(0x0400) == 2.0 ** -14
    assert oracle.decode_f16(0x7C00) == np.inf


def test_decode_bf16_all_patterns_against_format_definition():
    bits = np.arange(65536, dtype=np.uint16)
    want = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    got = np.array([oracle.decode_bf16(int(b)) for b in bits])
    both_nan = np.isnan(want) & np.isnan(got)
    assert np.all((want == got) | both_nan)
    assert oracle.decode_bf16(0x3F80) == 1.0
    assert oracle.decode_bf16(0x4049) == 3.140625
    assert oracle.decode_bf16(0x0001) == 2.0 ** -133
    assert oracle.decode_bf16(0xFF80) == -np.inf


def test_encoders_round_to_nearest_even_and_roundtrip():
    # ties: halfway between two neighbours goes to the even one
    assert encode_f16(np.array([1 + 2.0 ** -11]))[0] == 0x3C00
    assert encode_f16(np.array([1 + 3 * 2.0 ** -11]))[0] == 0x3C02
    assert encode_f16(np.array([1 + 2.0 ** -11 + 2.0 ** -20]))[0] == 0x3C01
    assert encode_bf16(np.array([1 + 2.0 ** -8]))[0] == 0x3F80
    assert encode_bf16(np.array([1 + 3 * 2.0 ** -8]))[0] == 0x3F82
    assert encode_bf16(np.array([1 + 2.0 ** -8 + 2.0 ** -20]))[0] == 0x3F81
    # every finite pattern survives decode -> encode
    bits = np.arange(65536, dtype=np.uint16)
    for dt, enc in ((DTYPE_F16, encode_f16), (DTYPE_BF16, encode_bf16)):
        v = decode_16(bits, dt)
        fin = np.isfinite(v)
        assert np.array_equal(enc(v[fin]), bits[fin])


def test_encoders_agree_with_torch_cast():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.standard_normal(20000), rng.uniform(-1, 1, 20000) * 1e-3,
                        rng.standard_normal(2000) * 300]).astype(np.float32)
    t = torch.from_numpy(x)
    assert np.array_equal(encode_f16(x), t.to(torch.float16).view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(encode_bf16(x), t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


# ---------------------------------------------------------------- L0: hand-worked products

A22 = [[1, 2], [3, 4]]
B22 = [[5, 6], [7, 8]]


@pytest.mark.parametrize("acc", [ACC_F32, ACC_F32FMA, ACC_F64])
def test_l0_hand_worked_2x2_all_trans(acc):
    assert np.array_equal(l0(A22, B22, acc=acc), [[19, 22], [43, 50]])
    assert np.array_equal(l0(A22, B22, "T", "N", acc=acc), [[26, 30], [38, 44]])
    assert np.array_equal(l0(A22, B22, "N", "T", acc=acc), [[17, 23], [39, 53]])
    assert np.array_equal(l0(A22, B22, "T", "T", acc=acc), [[23, 31], [34, 46]])
    # alpha = 2, beta = -1, C0 = ones: 2*AB - 1
    assert np.array_equal(l0(A22, B22, alpha=2, beta=-1, C0=np.ones((2, 2)), acc=acc), [[37, 43], [85, 99]])


@pytest.mark.parametrize("acc", [ACC_F32, ACC_F32FMA, ACC_F64])
def test_l0_hand_worked_3x2x4_with_padding(acc):
    A = [[1, 0, 2, -1], [3, 1, 0, 2], [0, -2, 1, 1]]          # 3 x 4
    B = [[1, 2], [0, 1], [-1, 3], [2, 0]]                     # 4 x 2
    want = [[-3, 8], [7, 7], [1, 1]]
    assert np.array_equal(l0(A, B, acc=acc, lda=5, ldb=7), want)
    At = np.array(A).T
    Bt = np.array(B).T
    assert np.array_equal(l0(At, B, "T", "N", acc=acc, lda=6), want)
    assert np.array_equal(l0(A, Bt, "N", "T", acc=acc, ldb=3), want)
    assert np.array_equal(l0(At, Bt, "T", "T", acc=acc, lda=4, ldb=2), want)
    C0 = [[1, -1], [2, 0], [0.5, 4]]
    got = l0(A, B, alpha=-0.5, beta=2, C0=C0, acc=acc)
    assert np.array_equal(got, -0.5 * np.array(want) + 2 * np.array(C0))


# ---------------------------------------------------------------- L0: closed forms

@pytest.mark.parametrize("acc", [ACC_F32, ACC_F32FMA, ACC_F64])
@pytest.mark.parametrize("m,n,k", [(5, 7, 1), (3, 4, 100), (17, 2, 4099)])
def test_l0_all_ones_gives_k(acc, m, n, k):
    got = l0(np.ones((m, k)), np.ones((k, n)), acc=acc)
    assert np.array_equal(got, np.full((m, n), float(k)))


@pytest.mark.parametrize("acc", [ACC_F32, ACC_F32FMA, ACC_F64])
def test_l0_identity_returns_other_operand(acc):
    rng = np.random.default_rng(1)
    X = rng.uniform(-1, 1, (6, 6)).astype(np.float32)
    eye = np.eye(6)
    assert np.array_equal(l0(eye, X, alpha=1.0, acc=acc), X)
    assert np.array_equal(l0(X, eye, alpha=1.0, acc=acc), X)
    # alpha a power of two: exact scaling
    assert np.array_equal(l0(eye, X, alpha=0.25, acc=acc), 0.25 * X)
    assert np.array_equal(l0(X, eye, "T", "N", alpha=-2.0, acc=acc), -2.0 * X.T)


@pytest.mark.parametrize("acc", [ACC_F32, ACC_F32FMA, ACC_F64])
def test_l0_beta_only_updates(acc):
    rng = np.random.default_rng(2)
    A = rng.uniform(-1, 1, (4, 3))
    B = rng.uniform(-1, 1, (3, 5))
    C0 = rng.uniform(-1, 1, (4, 5)).astype(np.float32)
    assert np.array_equal(l0(A, B, alpha=0.0, beta=1.0, C0=C0, acc=acc), C0)          # unchanged bitwise
    assert np.array_equal(l0(A, B, alpha=0.0, beta=0.5, C0=C0, acc=acc), 0.5 * C0)
    # k == 0: empty sum
    assert np.array_equal(l0(np.zeros((4, 0)), np.zeros((0, 5)), alpha=3.0, beta=-1.0, C0=C0, acc=acc), -C0)
    # beta == 0: C0 is never read (here it is NaN)
    got = l0(A, B, alpha=1.0, beta=0.0, C0=np.full((4, 5), np.nan), acc=acc)
    assert np.all(np.isfinite(got))


@pytest.mark.parametrize("acc", [ACC_F32, ACC_F32FMA, ACC_F64])
def test_l0_transpose_identity_bitwise(acc):
    # (A B)^T = B^T A^T: same products summed in the same k order, so bitwise equal
    rng = np.random.default_rng(3)
    A = rng.uniform(-1, 1, (7, 33)).astype(np.float32)
    B = rng.uniform(-1, 1, (33, 5)).astype(np.float32)
    C1 = l0(A, B, acc=acc)
    C2 = l0(B, A, "T", "T", acc=acc)      # op(B) = B^T (5 x 33), op(A) = A^T (33 x 7)
    assert np.array_equal(C1.T, C2)


@pytest.mark.parametrize("ta,tb", list(itertools.product("NT", "NT")))
def test_l0_f64_matches_library_matmul(ta, tb):
    rng = np.random.default_rng(4)
    m, n, k = 13, 9, 21
    A = rng.uniform(-1, 1, (m, k) if ta == "N" else (k, m)).astype(np.float32)
    B = rng.uniform(-1, 1, (k, n) if tb == "N" else (n, k)).astype(np.float32)
    C0 = rng.uniform(-1, 1, (m, n)).astype(np.float32)
    opA = A if ta == "N" else A.T
    opB = B if tb == "N" else B.T
    want = 1.5 * opA.astype(np.float64) @ opB.astype(np.float64) + 0.5 * C0
    got = l0(A, B, ta, tb, 1.5, 0.5, C0, lda=A.shape[0] + 3, ldb=B.shape[0] + 1)
    assert np.max(np.abs(got - want)) < 1e-13
    got32 = l0(A, B, ta, tb, 1.5, 0.5, C0, acc=ACC_F32)
    assert np.max(np.abs(got32 - want)) <= oracle.fp32_tolerance(k, 1.5, 0.5, 1, 1, 1)


def test_l0_f32_modes_round_like_float32():
    # 2^24 + 1 is not an fp32 number: summing 2^24 ones then one more stays at 2^24 in fp32, not in fp64
    k = 2 ** 24 + 1
    a = np.ones((1, k), dtype=np.float32)
    b = np.ones((k, 1), dtype=np.float32)
    assert l0(a, b, acc=ACC_F32)[0, 0] == 2.0 ** 24
    assert l0(a, b, acc=ACC_F64)[0, 0] == 2.0 ** 24 + 1
    # x = 1 + 2^-12: x*x = 1 + 2^-11 + 2^-24 needs 25 bits.  A separate multiply rounds it (tie to even)
    # to 1 + 2^-11 before the -1 is added; a fused multiply-add keeps the 2^-24.
    x = np.float32(1 + 2.0 ** -12)
    A = np.array([[1.0, x]], dtype=np.float32)
    B = np.array([[-1.0], [x]], dtype=np.float32)            # -1 + x*x, summed in that order
    assert l0(A, B, acc=ACC_F32)[0, 0] == 2.0 ** -11
    assert l0(A, B, acc=ACC_F32FMA)[0, 0] == 2.0 ** -11 + 2.0 ** -24
    assert l0(A, B, acc=ACC_F64)[0, 0] == 2.0 ** -11 + 2.0 ** -24


def test_l0_half_inputs_decoded_exactly():
    for dt, enc in ((OR_F16, encode_f16), (OR_BF16, encode_bf16)):
        A = make_matrix(5, 8, kind="normal", seed=9, matrix_id=0, dtype=dt, ld=6)
        B = make_matrix(8, 3, kind="normal", seed=9, matrix_id=1, dtype=dt, ld=11)
        c0 = np.zeros(15, dtype=np.float32)
        got = oracle.gemm_l0(dt, "N", "N", 5, 3, 8, 1.0, A.buf, A.ld, B.buf, B.ld, 0.0, c0, 5)
        want = A.as_f64() @ B.as_f64()
        assert np.max(np.abs(got - want)) < 1e-13


# ---------------------------------------------------------------- packing layout (Section III-A)

@pytest.mark.parametrize("ta", "NT")
def test_pack_A_layout_and_zero_padding(ta):
    m, k, mr = 21, 9, 8
    rows, cols = (m, k) if ta == "N" else (k, m)
    A = make_matrix(rows, cols, kind="index", seed=0, matrix_id=0, ld=rows + 2)
    opA = A.as_f64() if ta == "N" else A.as_f64().T
    ic, pc, mcb, kcb = 3, 2, 17, 6
    P = oracle.pack_A_f32(OR_F32, ta, A.buf, A.ld, ic, pc, mcb, kcb, mr)
    assert P.shape == (3, kcb, mr)                      # ceil(17/8) panels, each [kc][mr]
    for r in range(3):
        for p in range(kcb):
            for i in range(mr):
                row = r * mr + i
                want = opA[ic + row, pc + p] if row < mcb else 0.0
                assert P[r, p, i] == want


@pytest.mark.parametrize("tb", "NT")
def test_pack_B_layout_and_zero_padding(tb):
    k, n, nr = 10, 29, 12
    rows, cols = (k, n) if tb == "N" else (n, k)
    B = make_matrix(rows, cols, kind="index", seed=0, matrix_id=1, ld=rows + 1)
    opB = B.as_f64() if tb == "N" else B.as_f64().T
    pc, jc, kcb, ncb = 1, 2, 7, 26
    P = oracle.pack_B_f32(OR_F32, tb, B.buf, B.ld, pc, jc, kcb, ncb, nr)
    assert P.shape == (3, kcb, nr)
    for r in range(3):
        for p in range(kcb):
            for j in range(nr):
                col = r * nr + j
                want = opB[pc + p, jc + col] if col < ncb else 0.0
                assert P[r, p, j] == want


# ---------------------------------------------------------------- micro-kernel (Fig. 3 / Fig. 4)

def fig3_steps(mr, nr, kc, alpha, Ac, Bc, beta, C):
    """The four steps of the micro-kernel with alpha and beta in float32, spelled with scalar loops."""
    f = np.float32
    Cb = np.zeros((nr, mr), dtype=f)
    Ba = np.zeros((kc, nr), dtype=f)
    for cj in range(nr):
        for ci in range(mr):
            Cb[cj, ci] = f(C[cj, ci] * f(beta))
    for bk in range(kc):
        for bj in range(nr):
            Ba[bk, bj] = f(Bc[bk, bj] * f(alpha))
    for k in range(kc):
        for j in range(nr):
            for i in range(mr):
                Cb[j, i] = f(Cb[j, i] + f(Ac[k, i] * Ba[k, j]))
    return Cb


@pytest.mark.parametrize("mr,nr", [(8, 12), (4, 4), (1, 8), (8, 4)])
def test_ukernel_paper_order_matches_scalar_steps(mr, nr):
    rng = np.random.default_rng(7)
    kc = 19
    Ac = rng.uniform(-1, 1, (kc, mr)).astype(np.float32)
    Bc = rng.uniform(-1, 1, (kc, nr)).astype(np.float32)
    C = rng.uniform(-1, 1, (nr, mr)).astype(np.float32)
    got = oracle.ukernel_f32(mr, nr, kc, 1.5, Ac, Bc, 0.5, C, paper_scaling=True)
    assert np.array_equal(got, fig3_steps(mr, nr, kc, 1.5, Ac, Bc, 0.5, C))


def test_ukernel_rank_k_update_closed_forms():
    mr, nr, kc = 8, 12, 512
    ones_a = np.ones((kc, mr), dtype=np.float32)
    ones_b = np.ones((kc, nr), dtype=np.float32)
    C = np.arange(nr * mr, dtype=np.float32).reshape(nr, mr)
    for paper in (False, True):
        # alpha = beta = 1 (Fig. 4): C += Ac^T-outer-products = C + kc
        assert np.array_equal(oracle.ukernel_f32(mr, nr, kc, 1, ones_a, ones_b, 1, C, paper), C + kc)
        # one nonzero k slice: a single outer product a b^T, stored as C[j, i]
        Ac = np.zeros((kc, mr), dtype=np.float32)
        Bc = np.zeros((kc, nr), dtype=np.float32)
        Ac[37] = np.arange(1, mr + 1)
        Bc[37] = np.arange(1, nr + 1) * 10
        got = oracle.ukernel_f32(mr, nr, kc, 2, Ac, Bc, 0, C, paper)
        assert np.array_equal(got, 2 * np.outer(Bc[37], Ac[37]))


def test_ukernel_two_alpha_placements_agree():
    rng = np.random.default_rng(8)
    mr, nr, kc = 8, 12, 64
    Ai = rng.integers(-4, 5, (kc, mr)).astype(np.float32)
    Bi = rng.integers(-4, 5, (kc, nr)).astype(np.float32)
    Ci = rng.integers(-4, 5, (nr, mr)).astype(np.float32)
    # integer data, dyadic scalars: both placements of alpha are exact, hence identical
    a = oracle.ukernel_f32(mr, nr, kc, 1.5, Ai, Bi, 0.5, Ci, False)
    b = oracle.ukernel_f32(mr, nr, kc, 1.5, Ai, Bi, 0.5, Ci, True)
    assert np.array_equal(a, b)
    # random data: they differ only by rounding, inside the fp32 bound
    Ar = rng.uniform(-1, 1, (kc, mr)).astype(np.float32)
    Br = rng.uniform(-1, 1, (kc, nr)).astype(np.float32)
    Cr = rng.uniform(-1, 1, (nr, mr)).astype(np.float32)
    a = oracle.ukernel_f32(mr, nr, kc, 1.3, Ar, Br, 0.7, Cr, False)
    b = oracle.ukernel_f32(mr, nr, kc, 1.3, Ar, Br, 0.7, Cr, True)
    assert np.max(np.abs(a - b)) <= oracle.fp32_tolerance(kc, 1.3, 0.7, 1, 1, 1)


# ---------------------------------------------------------------- L1 (blocked, packed) against L0

def run_pair(m, n, k, ta, tb, alpha, beta, kind, seed, acc, pads=(0, 0, 0), dtype=DTYPE_F32, **blk):
    ar, ac = (m, k) if ta == "N" else (k, m)
    br, bc = (k, n) if tb == "N" else (n, k)
    A = make_matrix(ar, ac, kind=kind, seed=seed, matrix_id=0, dtype=dtype, ld=max(1, ar) + pads[0])
    B = make_matrix(br, bc, kind=kind, seed=seed, matrix_id=1, dtype=dtype, ld=max(1, br) + pads[1])
    C0 = make_matrix(m, n, kind=kind, seed=seed, matrix_id=2, ld=max(1, m) + pads[2])
    args = (dtype, ta, tb, m, n, k, alpha, A.buf, A.ld, B.buf, B.ld, beta, C0.buf, C0.ld)
    return oracle.gemm_l0(*args, acc=acc), oracle.gemm_l1(*args, acc=acc, **blk), (A, B, C0)


TINY = dict(mr=4, nr=4, mc=8, kc=4, nc=12)


def test_l1_bit_exact_on_integers_exhaustive_tiny_grid():
    # every (m, n, k) in 1..13 straddles mr, nr, mc, kc, nc of the tiny blocking at least once
    for m, n, k in itertools.product(range(1, 14), repeat=3):
        r0, r1, _ = run_pair(m, n, k, "N", "N", 1.5, 0.5, "int", 100 + m, ACC_F32, **TINY)
        assert np.array_equal(r0, r1), (m, n, k)


@pytest.mark.parametrize("ta,tb", list(itertools.product("NT", "NT")))
@pytest.mark.parametrize("blk", [TINY, dict(mr=8, nr=12, mc=16, kc=8, nc=24), dict(mr=1, nr=8, mc=5, kc=3, nc=8)])
def test_l1_bit_exact_on_integers_trans_and_padding(ta, tb, blk):
    for (m, n, k) in [(13, 25, 9), (37, 11, 30), (8, 12, 8), (1, 1, 1), (50, 3, 17)]:
        for alpha, beta in [(1, 0), (1.5, 0.5), (-1, 1)]:
            r0, r1, _ = run_pair(m, n, k, ta, tb, alpha, beta, "int", 7, ACC_F32, pads=(1, 2, 3), **blk)
            assert np.array_equal(r0, r1)
            r0, r1, _ = run_pair(m, n, k, ta, tb, alpha, beta, "int", 7, ACC_F64, pads=(1, 2, 3), **blk)
            assert np.array_equal(r0, r1)


@pytest.mark.parametrize("ta,tb", list(itertools.product("NT", "NT")))
def test_l1_equals_l0_bitwise_when_k_fits_one_block(ta, tb):
    # k <= kc: the blocked algorithm sums each entry in the same order as the definition
    r0, r1, _ = run_pair(45, 53, 64, ta, tb, 1.5, 0.5, "uniform", 11, ACC_F32, mr=8, nr=12, mc=24, kc=64, nc=36)
    assert np.array_equal(r0, r1)
    r0, r1, _ = run_pair(45, 53, 512, ta, tb, 1.0, 0.0, "uniform", 12, ACC_F32)
    assert np.array_equal(r0, r1)


def test_l1_random_within_fp32_bound_default_blocking():
    m, n, k = 150, 130, 1300     # several kc blocks, ragged mc / nc / mr / nr edges
    r64, _, (A, B, C0) = run_pair(m, n, k, "N", "N", 1.5, 0.5, "uniform", 13, ACC_F64)
    _, r1, _ = run_pair(m, n, k, "N", "N", 1.5, 0.5, "uniform", 13, ACC_F32)
    tol = oracle.fp32_tolerance(k, 1.5, 0.5, A.max_abs(), B.max_abs(), C0.max_abs())
    assert np.max(np.abs(r1 - r64)) <= tol


def test_l1_paper_scaling_mode_within_bound_and_exact_on_integers():
    m, n, k = 40, 36, 70
    A = make_matrix(m, k, kind="uniform", seed=21, matrix_id=0)
    B = make_matrix(k, n, kind="uniform", seed=21, matrix_id=1)
    C0 = make_matrix(m, n, kind="uniform", seed=21, matrix_id=2)
    args = (OR_F32, "N", "N", m, n, k, 1.3, A.buf, A.ld, B.buf, B.ld, 0.7, C0.buf, C0.ld)
    ref = oracle.gemm_l0(*args, acc=ACC_F64)
    got = oracle.gemm_l1(*args, acc=ACC_F32, paper_scaling=True, mr=8, nr=12, mc=16, kc=32, nc=24)
    assert np.max(np.abs(got - ref)) <= oracle.fp32_tolerance(k, 1.3, 0.7, 1, 1, 1)
    Ai = make_matrix(m, k, kind="int", seed=22, matrix_id=0)
    Bi = make_matrix(k, n, kind="int", seed=22, matrix_id=1)
    Ci = make_matrix(m, n, kind="int", seed=22, matrix_id=2)
    args = (OR_F32, "N", "N", m, n, k, 1.5, Ai.buf, Ai.ld, Bi.buf, Bi.ld, 0.5, Ci.buf, Ci.ld)
    assert np.array_equal(oracle.gemm_l0(*args, acc=ACC_F32),
                          oracle.gemm_l1(*args, acc=ACC_F32, paper_scaling=True, mr=8, nr=12, mc=16, kc=32, nc=24))


def test_l1_beta_zero_never_reads_c_and_k_zero():
    m, n, k = 9, 7, 5
    A = make_matrix(m, k, kind="uniform", seed=1, matrix_id=0)
    B = make_matrix(k, n, kind="uniform", seed=1, matrix_id=1)
    nanC = np.full(m * n, np.nan, dtype=np.float32)
    got = oracle.gemm_l1(OR_F32, "N", "N", m, n, k, 1.0, A.buf, m, B.buf, k, 0.0, nanC, m, **TINY)
    assert np.all(np.isfinite(got))
    C0 = make_matrix(m, n, kind="uniform", seed=1, matrix_id=2)
    got = oracle.gemm_l1(OR_F32, "N", "N", m, n, 0, 1.0, A.buf, m, B.buf, 1, 0.5, C0.buf, m, **TINY)
    assert np.array_equal(got, 0.5 * C0.as_f64())


def test_l1_f64_half_inputs_match_library_matmul():
    for dt in (DTYPE_F16, DTYPE_BF16):
        m, n, k = 33, 47, 700
        A = make_matrix(m, k, kind="normal", seed=3, matrix_id=0, dtype=dt)
        B = make_matrix(k, n, kind="normal", seed=3, matrix_id=1, dtype=dt)
        c0 = np.zeros(m * n, dtype=np.float32)
        got = oracle.gemm_l1(dt, "N", "N", m, n, k, 1.0, A.buf, m, B.buf, k, 0.0, c0, m, acc=ACC_F64)
        want = A.as_f64() @ B.as_f64()
        assert np.linalg.norm(got - want) / np.linalg.norm(want) < 1e-14


# ---------------------------------------------------------------- sampled entries and the randomised check

def test_samples_match_library_matmul():
    m, n, k = 31, 29, 200
    A = make_matrix(k, m, kind="uniform", seed=5, matrix_id=0, ld=k + 4)       # transA = T
    B = make_matrix(k, n, kind="uniform", seed=5, matrix_id=1)
    C0 = make_matrix(m, n, kind="uniform", seed=5, matrix_id=2, ld=m + 1)
    want = 1.5 * A.as_f64().T @ B.as_f64() + 0.5 * C0.as_f64()
    rows = np.array([0, 30, 0, 30, 7, 19])
    cols = np.array([0, 28, 28, 0, 3, 11])
    got = oracle.gemm_samples_f64(OR_F32, "T", "N", k, 1.5, A.buf, A.ld, B.buf, B.ld, 0.5, C0.buf, C0.ld, rows, cols)
    assert np.max(np.abs(got - want[rows, cols])) < 1e-12


def test_freivalds_accepts_exact_product_and_finds_planted_error():
    m, n, k = 64, 48, 96
    A = make_matrix(m, k, kind="int", seed=6, matrix_id=0)
    B = make_matrix(n, k, kind="int", seed=6, matrix_id=1)                    # transB = T
    C0 = make_matrix(m, n, kind="int", seed=6, matrix_id=2)
    want = (2.0 * A.as_f64() @ B.as_f64().T - C0.as_f64()).astype(np.float32)   # exact in fp32
    C, ldc = colmajor(want, m + 5)
    rng = np.random.default_rng(0)
    x = rng.choice([-1.0, 1.0], n)
    args = (OR_F32, "N", "T", m, n, k, 2.0, A.buf, A.ld, B.buf, B.ld, -1.0, C0.buf, C0.ld)
    resid, scale = oracle.freivalds(*args, C, ldc, x)
    assert np.all(resid == 0.0) and np.all(scale > 0)
    C[17 + 5 * ldc] += 3.0                                                      # plant one wrong entry
    resid, _ = oracle.freivalds(*args, C, ldc, x)
    assert abs(resid[17]) == 3.0 and np.count_nonzero(resid) == 1


# ---------------------------------------------------------------- shapes of the lowered convolutions

def read_table(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append(tuple(int(t) for t in line.split()))
    return rows


def test_resnet50_shapes_reproduce_paper_table():
    table = read_table("resnet50_v15_im2row_batch1.txt")
    assert len(table) == 20
    got = im2row_shapes(RESNET50_V15_BATCH1, batch=1, weights_as_A=False)
    assert [(i + 1, *s) for i, s in enumerate(got)] == table
    # the first layer is the edge case the text names: 12544 x 64 x 147
    assert got[0] == (12544, 64, 147)
    # batch 32 with weights as operand A: m <- channels, n <- 32 * pixels
    b32 = im2row_shapes(RESNET50_V15_BATCH1, batch=32, weights_as_A=True)
    assert b32[2] == (64, 32 * 56 * 56, 64 * 3 * 3)
    assert b32[6] == (128, 32 * 28 * 28, 128 * 3 * 3)
    assert b32[11] == (256, 32 * 14 * 14, 256 * 3 * 3)
    assert b32[16] == (512, 32 * 7 * 7, 512 * 3 * 3)


def test_vgg16_shapes_reproduce_paper_table():
    table = read_table("vgg16_im2row_batch1.txt")
    got = im2row_shapes(VGG16_BATCH1, batch=1, weights_as_A=False)
    assert [(i + 1, *s) for i, s in enumerate(got)] == table


# ---------------------------------------------------------------- binary16 accumulation (the paper's f16 arithmetic)

def test_round_f16_fixed_points_ties_and_library_conversion():
    # every binary16 number is its own rounding; the midpoint of two neighbours goes to the one with an even last bit
    pats = np.arange(0, 0x7C00, dtype=np.uint16)                       # all non-negative finite patterns, in increasing order
    vals = pats.view(np.float16).astype(np.float64)
    for step in (1, 37, 401):                                           # a few thousand of them, spread over all exponents
        for i in range(0, len(vals) - 1, step):
            assert oracle.round_f16(vals[i]) == vals[i]
            mid = 0.5 * (vals[i] + vals[i + 1])                         # exact in double
            even = vals[i] if (int(pats[i]) & 1) == 0 else vals[i + 1]
            assert oracle.round_f16(mid) == even, (i, mid)
            assert oracle.round_f16(-mid) == -even
    # against the library's conversion (other code) on random values of all magnitudes, overflow included
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(4000) * 10.0 ** rng.integers(-9, 6, 4000), [65519.9, 65520.0, 70000.0, 1e-8, 2.0 ** -25, 3 * 2.0 ** -26]])
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).astype(np.float64)
    got = np.array([oracle.round_f16(v) for v in x])
    assert np.array_equal(got, want)


def test_l0_binary16_accumulation_rounds_the_running_sum():
    # 2048 + 1 + 1: in binary16 the spacing at 2048 is 2, so each +1 is a tie that goes back to 2048 (even); fp32 gives 2050
    A = Matrix(encode_f16(np.array([2048.0, 1.0, 1.0])), 1, 3, 1, DTYPE_F16)
    B = Matrix(encode_f16(np.array([1.0, 1.0, 1.0])), 3, 1, 3, DTYPE_F16)
    C0 = np.zeros(1, dtype=np.float32)
    args = (DTYPE_F16, "N", "N", 1, 1, 3, 1.0, A.buf, 1, B.buf, 3, 0.0, C0, 1)
    assert oracle.gemm_l0(*args, acc=oracle.ACC_F16)[0, 0] == 2048.0
    assert oracle.gemm_l0(*args, acc=ACC_F32)[0, 0] == 2050.0
    # the same sum started from the small terms is exact: 1 + 1 + 2048 = 2050
    A2 = Matrix(encode_f16(np.array([1.0, 1.0, 2048.0])), 1, 3, 1, DTYPE_F16)
    assert oracle.gemm_l0(DTYPE_F16, "N", "N", 1, 1, 3, 1.0, A2.buf, 1, B.buf, 3, 0.0, C0, 1, acc=oracle.ACC_F16)[0, 0] == 2050.0
    # random data against a scalar loop in the library's binary16 type (its conversion from double rounds once, to nearest even)
    rng = np.random.default_rng(5)
    m, n, k = 7, 5, 300
    a = rng.standard_normal((m, k)).astype(np.float16)
    b = rng.standard_normal((k, n)).astype(np.float16)
    c0 = rng.standard_normal((m, n)).astype(np.float32)
    want = np.zeros((m, n))
    for i in range(m):
        for j in range(n):
            s = np.float16(0)
            for p in range(k):
                s = np.float16(np.float64(s) + np.float64(a[i, p]) * np.float64(b[p, j]))
            want[i, j] = 1.5 * np.float64(s) + 0.5 * np.float64(c0[i, j])
    got = oracle.gemm_l0(DTYPE_F16, "N", "N", m, n, k, 1.5, np.ascontiguousarray(a.T).ravel().view(np.uint16), m,
                         np.ascontiguousarray(b.T).ravel().view(np.uint16), k, 0.5, np.ascontiguousarray(c0.T).ravel(), m,
                         acc=oracle.ACC_F16)
    assert np.array_equal(got, want)
    # integer data whose partial sums are all binary16 numbers: identical to the fp64 mode
    ai = rng.integers(-4, 5, (m, 64)).astype(np.float16)
    bi = rng.integers(-4, 5, (64, n)).astype(np.float16)
    pa, pb = np.ascontiguousarray(ai.T).ravel().view(np.uint16), np.ascontiguousarray(bi.T).ravel().view(np.uint16)
    z = np.zeros(m * n, dtype=np.float32)
    assert np.array_equal(oracle.gemm_l0(DTYPE_F16, "N", "N", m, n, 64, 1.0, pa, m, pb, 64, 0.0, z, m, acc=oracle.ACC_F16),
                          oracle.gemm_l0(DTYPE_F16, "N", "N", m, n, 64, 1.0, pa, m, pb, 64, 0.0, z, m, acc=ACC_F64))
