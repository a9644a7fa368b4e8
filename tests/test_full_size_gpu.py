"""Parity at the full sizes of the workloads, in the configuration the selector picks for them (the one
bench.py times).  The CPU oracle cannot compute whole results of this size in reasonable time, so each
result is checked (a) over the whole matrix by a randomised fp64 identity (C x against alpha A (B x) + beta C0 x
for +-1 probe vectors) and (b) entry by entry against exact fp64 dot products on corners, tile-edge positions,
thousands of scattered entries and sampled full rows and columns; integer-valued runs are compared bitwise on
the sampled entries."""
import numpy as np
import pytest

import oracle
import paper_2310_17408_b200 as g
from workloads import DTYPE_BF16, DTYPE_F16, DTYPE_F32, config_problems

from gpu_util import check_large, run_problem, sample_positions

pytestmark = pytest.mark.gpu


def run_and_check(p, seed=0):
    A, B, C0 = p.operands()
    C, cfg = run_problem(p, A, B, C0, check_inputs=False)
    err = check_large(p, A, B, C0, C, cfg, seed=seed)
    return cfg, err


def test_config1_512_full_oracle_and_integer_bit_exact():
    from gpu_util import check_against_oracle
    p = config_problems(1)[0]
    A, B, C0 = p.operands()
    C, cfg = run_problem(p, A, B, C0)
    check_against_oracle(p, A, B, C0, C)
    p = config_problems(1, integer=True)[0]
    A, B, C0 = p.operands()
    C, cfg = run_problem(p, A, B, C0)
    check_against_oracle(p, A, B, C0, C, integer=True)


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_config2_square_fp32_sweep(idx):
    p = config_problems(2)[idx]
    cfg, _ = run_and_check(p, seed=idx)
    assert cfg["kernel"] == g.GEMM_KERNEL_SIMT_FAST


def test_config3_im2row_fp32_all_layers():
    for i, p in enumerate(config_problems(3)):
        cfg, _ = run_and_check(p, seed=i)
        assert cfg["kernel"] == g.GEMM_KERNEL_SIMT_FAST, (p.name, cfg)


def test_config4_nonsquarish_fp32():
    for i, p in enumerate(config_problems(4)):
        cfg, _ = run_and_check(p, seed=i)
        assert cfg["kernel"] == g.GEMM_KERNEL_SIMT_FAST
    assert cfg["split_k"] > 1          # 256 x 256 x 65536: split-k is mandatory


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_config5_half_squares_4096_8192(dtype):
    for i, p in enumerate(config_problems(5, dtype=dtype)[:2]):
        cfg, _ = run_and_check(p, seed=i)
        assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR
        assert (cfg["tile_m"], cfg["tile_n"]) == (256, 256)      # large squares run on CTA pairs


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_config5_half_square_16384(dtype):
    p = config_problems(5, dtype=dtype)[2]
    cfg, _ = run_and_check(p)
    assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR
    assert (cfg["tile_m"], cfg["tile_n"]) == (256, 256)


@pytest.mark.parametrize("dtype", [DTYPE_F16, DTYPE_BF16])
def test_config5_half_im2row_all_layers(dtype):
    for i, p in enumerate(config_problems(5, dtype=dtype)[3:]):
        cfg, _ = run_and_check(p, seed=i)
        assert cfg["kernel"] == g.GEMM_KERNEL_TENSOR, (p.name, cfg)


def test_full_size_members_with_alpha_and_beta():
    # the workloads are timed at alpha = 1, beta = 0; one member of each of configs 3, 4 and 5 is also checked at
    # full size with alpha = 1.5, beta = 0.5 and a pre-filled C (the epilogue then reads C)
    import dataclasses
    cases = [config_problems(3)[2], config_problems(4)[0], config_problems(4)[3],
             config_problems(5, dtype=DTYPE_BF16)[1], config_problems(5, dtype=DTYPE_F16)[9]]
    for i, p in enumerate(cases):
        q = dataclasses.replace(p, name=p.name + "_ab", alpha=1.5, beta=0.5)
        cfg, _ = run_and_check(q, seed=100 + i)


def test_integer_valued_large_shapes_bit_exact_on_samples():
    # integer entries in [-4, 4]: every partial sum is exact in fp32, so sampled entries must match bitwise
    cases = [config_problems(2, integer=True)[2], config_problems(4, integer=True)[3],
             config_problems(5, integer=True, dtype=DTYPE_BF16)[0], config_problems(5, integer=True, dtype=DTYPE_F16)[5]]
    for p in cases:
        A, B, C0 = p.operands()
        C, cfg = run_problem(p, A, B, C0, check_inputs=False)
        rng = np.random.default_rng(1)
        rows, cols = sample_positions(p.m, p.n, cfg["tile_m"], cfg["tile_n"], rng, scattered=2048)
        ref = oracle.gemm_samples_f64(p.dtype, p.transA, p.transB, p.k, p.alpha, A.buf, A.ld, B.buf, B.ld, p.beta,
                                      C0.buf, C0.ld, rows, cols)
        got = C.window()[rows, cols]
        assert np.array_equal(got.astype(np.float64), ref), p.name


def test_vgg16_and_paper_orientation_shapes():
    # second workload (VGG16 at batch 32, includes k = 27) and the tall-and-skinny orientation the paper's tables use
    from workloads import im2row_problems
    vgg, px = im2row_problems("vgg16"), im2row_problems("resnet50", weights_as_A=False)
    cases = [vgg[0], vgg[6], im2row_problems("vgg16", dtype=DTYPE_BF16)[0], px[0], px[6], px[16],
             im2row_problems("resnet50", weights_as_A=False, dtype=DTYPE_F16)[0],
             im2row_problems("resnet50", weights_as_A=False, dtype=DTYPE_BF16)[11],
             im2row_problems("vgg16", weights_as_A=False)[8]]
    for i, p in enumerate(cases):
        run_and_check(p, seed=i)


@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_BF16])
def test_result_with_more_than_2_31_entries(dtype):
    # C has 32768 x 65600 = 2.15e9 entries (8.6 GB): every index into C must be 64-bit.  beta = 0, so C is
    # allocated on the device only; sampled columns (first, last, around the 2^31-entry mark) are checked exactly.
    import torch
    from workloads import make_matrix
    from gpu_util import to_device
    m, n, k = 32768, 65600, 32
    A = make_matrix(m, k, kind="int", seed=77, matrix_id=0, dtype=dtype)
    B = make_matrix(k, n, kind="int", seed=77, matrix_id=1, dtype=dtype)
    dA, dB = to_device(A), to_device(B)
    dC = torch.full((m * n,), float("nan"), dtype=torch.float32, device="cuda")
    rc = g.gemm(dtype, "N", "N", m, n, k, 1.0, dA.data_ptr(), m, dB.data_ptr(), k, 0.0, dC.data_ptr(), m,
                torch.cuda.current_stream().cuda_stream)
    assert rc == 0, g.gemm_status_string(rc)
    assert g.gemm_poll_status() == 0
    cols = [0, 1, 255, 256, 65535, 65536, 65537, n - 257, n - 2, n - 1]       # 65536 * 32768 = 2^31 entries
    ref = A.as_f64() @ B.as_f64()[:, cols]
    got = torch.stack([dC[j * m:(j + 1) * m] for j in cols], dim=1).cpu().numpy().astype(np.float64)
    assert np.array_equal(got, ref)
    # nothing left unwritten anywhere: no NaN survives in the whole result
    assert not bool(torch.isnan(dC).any())
    del dC
    torch.cuda.empty_cache()


def test_gemm_host_at_the_end_to_end_size_of_the_bench():
    # config 2's largest member through the host-buffer entry point, as bench.py's e2e leg calls it (pinned buffers,
    # alpha = 1.5, beta = 0.5): eight k panels of A, leading column panels joining one by one, the first panel and the
    # first k panel cut in two.  Different summation order than gemm(), same bound.
    import torch
    p = config_problems(2)[3]
    A, B, C0 = p.operands()
    C = C0.copy()
    pinned = [torch.from_numpy(x.buf).pin_memory() for x in (A, B, C)]
    rc = g.gemm_host(p.api_dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, pinned[0].data_ptr(), A.ld, pinned[1].data_ptr(),
                     B.ld, p.beta, pinned[2].data_ptr(), C.ld, torch.cuda.current_stream().cuda_stream)
    assert rc == 0, g.gemm_status_string(rc)
    assert g.gemm_poll_status() == 0
    C.buf[:] = pinned[2].numpy()
    cfg = g.gemm_last_config()
    check_large(p, A, B, C0, C, cfg, seed=11)
