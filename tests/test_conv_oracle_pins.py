"""Pins of the convolution oracle (oracle/conv_oracle.c) to things other than itself: a library convolution that
uses another tensor layout and other code, closed forms, special cases that reduce to a plain matrix product, and
the identity between the two routes the oracle offers (definition vs. im2row lowering followed by the GEMM oracle).
A dropped tap, a swapped stride or padding, a transposed filter index or a wrong patch order fails at least one."""
import numpy as np
import pytest
import torch

import oracle
from workloads import DTYPE_BF16, DTYPE_F16, DTYPE_F32, ConvProblem, conv_layer_problems, make_matrix

GEOMS = [
    # batch, h, w, c_in, c_out, kh, kw, stride, pad
    (2, 7, 9, 3, 5, 3, 3, 1, 1),
    (1, 12, 10, 4, 6, 7, 7, 2, 3),
    (3, 5, 5, 8, 4, 1, 1, 1, 0),
    (2, 9, 8, 2, 3, 3, 3, 2, 0),
    (1, 6, 6, 5, 2, 5, 5, 1, 2),
    (2, 4, 11, 6, 7, 3, 3, 3, 1),
]


def geom_of(p: ConvProblem):
    return oracle.conv_geom(p.batch, p.h, p.w, p.c_in, p.c_out, p.kh, p.kw, p.stride, p.stride, p.pad, p.pad)


def problem(g, dtype=DTYPE_F32, kind=None, alpha=1.0, beta=0.0, seed=3, ld_pad=(0, 0)):
    b, h, w, ci, co, kh, kw, st, pd = g
    kinds = dict(kindX=kind, kindW=kind, kindY=kind) if kind else {}
    return ConvProblem("t", dtype, b, h, w, ci, co, kh, kw, st, pd, alpha, beta, seed=seed, ld_pad=ld_pad, **kinds)


def torch_reference(p: ConvProblem, X, W, Y0):
    """Library routine on another layout: NCHW activations, (C_out, C_in, kh, kw) filters, fp64."""
    x = torch.from_numpy(X.as_f64().T.reshape(p.batch, p.h, p.w, p.c_in).transpose(0, 3, 1, 2).copy())
    wt = torch.from_numpy(W.as_f64().reshape(p.c_out, p.kh, p.kw, p.c_in).transpose(0, 3, 1, 2).copy())
    y = torch.nn.functional.conv2d(x, wt, stride=p.stride, padding=p.pad)            # (b, co, ho, wo)
    y = y.permute(1, 0, 2, 3).reshape(p.c_out, -1).numpy()
    return p.alpha * y + (p.beta * Y0.as_f64() if p.beta != 0.0 else 0.0)


@pytest.mark.parametrize("g", GEOMS)
@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_F16, DTYPE_BF16])
def test_direct_matches_library_convolution(g, dtype):
    p = problem(g, dtype, alpha=1.5, beta=0.5, ld_pad=(3, 2))
    X, W, Y0 = p.operands()
    got = oracle.conv2d_direct(dtype, geom_of(p), p.alpha, X.buf, W.buf, W.ld, p.beta, Y0.buf, Y0.ld)
    ref = torch_reference(p, X, W, Y0)
    assert got.shape == ref.shape == (p.c_out, p.gemm_mnk[1])
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("g", GEOMS)
def test_integer_inputs_match_library_exactly(g):
    p = problem(g, DTYPE_F32, kind="int")
    X, W, Y0 = p.operands()
    got = oracle.conv2d_direct(DTYPE_F32, geom_of(p), 1.0, X.buf, W.buf, W.ld)
    assert np.array_equal(got, torch_reference(p, X, W, Y0))


@pytest.mark.parametrize("g", GEOMS)
@pytest.mark.parametrize("dtype", [DTYPE_F32, DTYPE_BF16])
def test_lowering_then_gemm_oracle_equals_direct_bitwise(g, dtype):
    # the paper's route (im2row, then GEMM) and the definition add the same products in the same order
    p = problem(g, dtype, alpha=-0.75, beta=1.25, ld_pad=(1, 0))
    X, W, Y0 = p.operands()
    geo = geom_of(p)
    m, n, k = p.gemm_mnk
    low = oracle.im2row(dtype, geo, X.buf, ld=k + 2)
    via_gemm = oracle.gemm_l0(dtype, "N", "N", m, n, k, p.alpha, W.buf, W.ld, low, k + 2, p.beta, Y0.buf, Y0.ld,
                              acc=oracle.ACC_F64)
    direct = oracle.conv2d_direct(dtype, geo, p.alpha, X.buf, W.buf, W.ld, p.beta, Y0.buf, Y0.ld)
    assert np.array_equal(via_gemm, direct)


def test_lowered_matrix_layout_by_index_values():
    # activations that hold their own linear index: every entry of the lowered matrix can be predicted
    b, h, w, ci, kh, kw, st, pd = 2, 5, 6, 3, 3, 2, 2, 1
    p = ConvProblem("t", DTYPE_F32, b, h, w, ci, 4, kh, kw, st, pd, kindX="index")
    X, _, _ = p.operands()
    geo = oracle.conv_geom(b, h, w, ci, 4, kh, kw, st, st, pd, pd)
    ho, wo = oracle.conv_out_hw(geo)
    assert (ho, wo) == ((h + 2 * pd - kh) // st + 1, (w + 2 * pd - kw) // st + 1) == p.out_hw
    k = kh * kw * ci
    low = oracle.im2row(DTYPE_F32, geo, X.buf).reshape(b * ho * wo, k)
    for j in range(b * ho * wo):
        bb, oh, ow = j // (ho * wo), (j // wo) % ho, j % wo
        for r in range(kh):
            for s in range(kw):
                hi, wi = oh * st - pd + r, ow * st - pd + s
                for c in range(ci):
                    want = float(((bb * h + hi) * w + wi) * ci + c) if 0 <= hi < h and 0 <= wi < w else 0.0
                    assert low[j, (r * kw + s) * ci + c] == want


def test_all_ones_counts_the_taps_inside_the_image():
    b, h, w, ci, co, ks, pd = 1, 6, 7, 5, 3, 3, 1
    p = ConvProblem("t", DTYPE_F32, b, h, w, ci, co, ks, ks, 1, pd, kindX="ones", kindW="ones")
    X, W, _ = p.operands()
    got = oracle.conv2d_direct(DTYPE_F32, geom_of(p), 1.0, X.buf, W.buf, W.ld).reshape(co, h, w)
    rows = np.array([min(i + 1, h - 1) - max(i - 1, 0) + 1 for i in range(h)])
    cols = np.array([min(j + 1, w - 1) - max(j - 1, 0) + 1 for j in range(w)])
    want = ci * np.outer(rows, cols)              # 9 taps inside, 6 on an edge, 4 in a corner, times C_in
    for c in range(co):
        assert np.array_equal(got[c], want)


def test_one_by_one_layer_is_a_plain_matrix_product():
    p = problem((2, 4, 5, 6, 3, 1, 1, 1, 0), DTYPE_F32)
    X, W, _ = p.operands()
    got = oracle.conv2d_direct(DTYPE_F32, geom_of(p), 1.0, X.buf, W.buf, W.ld)
    np.testing.assert_allclose(got, W.as_f64() @ X.as_f64(), rtol=1e-13, atol=1e-13)


def test_delta_filter_shifts_the_image():
    # one tap (r, s) = (0, 2) of a 3 x 3 filter set to 1 on the diagonal channel pairs: Y(b, ho, wo, c) = X(b, ho-1, wo+1, c)
    b, h, w, c = 1, 5, 6, 4
    p = ConvProblem("t", DTYPE_F32, b, h, w, c, c, 3, 3, 1, 1, kindW="zeros")
    X, W, _ = p.operands()
    Wm = W.window()
    for ch in range(c):
        Wm[ch, (0 * 3 + 2) * c + ch] = 1.0
    got = oracle.conv2d_direct(DTYPE_F32, geom_of(p), 1.0, X.buf, W.buf, W.ld).reshape(c, h, w)
    x = X.as_f64().T.reshape(h, w, c)
    want = np.zeros((c, h, w))
    for oh in range(h):
        for ow in range(w):
            hi, wi = oh - 1, ow + 1
            if 0 <= hi < h and 0 <= wi < w:
                want[:, oh, ow] = x[hi, wi, :]
    assert np.array_equal(got, want)


def test_beta_zero_never_reads_the_previous_result_and_samples_agree():
    p = problem(GEOMS[0], DTYPE_F16, alpha=2.0, beta=0.0)
    X, W, Y0 = p.operands()
    Y0.buf[:] = np.nan
    full = oracle.conv2d_direct(DTYPE_F16, geom_of(p), 2.0, X.buf, W.buf, W.ld, 0.0, Y0.buf, Y0.ld)
    assert np.all(np.isfinite(full))
    rng = np.random.default_rng(0)
    rows, cols = rng.integers(0, full.shape[0], 50), rng.integers(0, full.shape[1], 50)
    got = oracle.conv2d_samples_f64(DTYPE_F16, geom_of(p), 2.0, X.buf, W.buf, W.ld, 0.0, None, 0, rows, cols)
    assert np.array_equal(got, full[rows, cols])


def test_layer_list_reproduces_the_lowered_gemm_dimensions_of_the_tables():
    import os
    from workloads import RESNET50_V15_BATCH1, VGG16_BATCH1, im2row_shapes
    here = os.path.dirname(__file__)
    for net, layers, fn in (("resnet50", RESNET50_V15_BATCH1, "resnet50_v15_im2row_batch1.txt"),
                            ("vgg16", VGG16_BATCH1, "vgg16_im2row_batch1.txt")):
        rows = [tuple(int(x) for x in ln.split()[1:]) for ln in open(os.path.join(here, "golden", fn)) if ln[0] != "#" and ln.strip()]
        probs = conv_layer_problems(net, batch=1)
        assert [(p.gemm_mnk[1], p.gemm_mnk[0], p.gemm_mnk[2]) for p in probs] == rows      # table: m = pixels, n = C_out
