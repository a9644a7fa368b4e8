"""The seeded input generators: determinism, independence of the leading dimension, value ranges."""
import numpy as np

from workloads import DTYPE_BF16, DTYPE_F16, DTYPE_F32, config_problems, make_matrix
from workloads.generators import raw_u64


def test_counter_mode_is_random_access():
    whole = raw_u64(3, 1, 0, 1000)
    assert np.array_equal(raw_u64(3, 1, 200, 50), whole[200:250])
    assert not np.array_equal(raw_u64(3, 2, 0, 1000), whole)
    assert not np.array_equal(raw_u64(4, 1, 0, 1000), whole)


def test_same_logical_matrix_for_any_ld_and_padding_is_canary():
    a = make_matrix(37, 11, kind="uniform", seed=5, matrix_id=0)
    b = make_matrix(37, 11, kind="uniform", seed=5, matrix_id=0, ld=48)
    assert np.array_equal(a.window(), b.window())
    assert b.padding().shape == (11, 11) and b.padding_intact()
    b.buf[40] = 1.0
    assert not b.padding_intact()


def test_value_distributions():
    u = make_matrix(512, 512, kind="uniform", seed=0, matrix_id=0).as_f64()
    assert u.min() >= -1.0 and u.max() < 1.0 and abs(u.mean()) < 0.01 and abs(u.var() - 1 / 3) < 0.01
    assert np.array_equal(u * 2 ** 23, np.round(u * 2 ** 23))          # on the 2^-23 grid
    z = make_matrix(512, 512, kind="normal", seed=0, matrix_id=1, scale=0.5).as_f64()
    assert abs(z.mean()) < 0.01 and abs(z.std() - 0.5) < 0.01
    r = make_matrix(512, 512, kind="absnormal", seed=0, matrix_id=1).as_f64()
    assert r.min() >= 0 and abs(r.mean() - np.sqrt(2 / np.pi)) < 0.01
    i = make_matrix(300, 300, kind="int", seed=0, matrix_id=2).as_f64()
    assert set(np.unique(i)) == set(range(-4, 5))
    for dt in (DTYPE_F16, DTYPE_BF16):
        ih = make_matrix(64, 64, kind="int", seed=0, matrix_id=2, dtype=dt).as_f64()
        assert np.array_equal(ih, make_matrix(64, 64, kind="int", seed=0, matrix_id=2).as_f64())


def test_config_lists():
    assert [(p.m, p.n, p.k) for p in config_problems(1)] == [(512, 512, 512)]
    assert config_problems(1)[0].seed == 0
    c2 = config_problems(2)
    assert [p.m for p in c2] == [1024, 2048, 4096, 8192] and all(p.alpha == 1.5 and p.beta == 0.5 for p in c2)
    c3 = config_problems(3)
    assert len(c3) == 20 and (c3[0].m, c3[0].n, c3[0].k) == (64, 32 * 112 * 112, 147)
    assert abs(c3[2].scaleA ** 2 - 2.0 / 576) < 1e-15
    c4 = config_problems(4)
    assert (c4[3].m, c4[3].n, c4[3].k) == (256, 256, 65536)
    c5 = config_problems(5, dtype=DTYPE_BF16)
    assert len(c5) == 23 and c5[0].dtype == DTYPE_BF16 and c5[2].m == 16384
    assert len({p.seed for p in c5}) == 23


def test_second_workload_and_paper_orientation():
    from workloads import im2row_problems
    v = im2row_problems("vgg16")
    assert len(v) == 9 and (v[0].m, v[0].n, v[0].k) == (64, 32 * 224 * 224, 27)
    px = im2row_problems("resnet50", weights_as_A=False)
    assert len(px) == 20 and (px[0].m, px[0].n, px[0].k) == (32 * 112 * 112, 64, 147)
    assert px[0].kindA == "absnormal" and px[0].kindB == "normal" and abs(px[0].scaleB ** 2 - 2 / 147) < 1e-15
    assert len({p.seed for p in v + px}) == 29


def test_sixteen_bit_result_variants_of_the_workloads():
    from workloads import DTYPE_BF16, config_problems, conv_layer_problems
    plain, c16 = config_problems(5, dtype=DTYPE_BF16), config_problems(5, dtype=DTYPE_BF16, c16=True)
    assert [p.name + "_c16" for p in plain] == [p.name for p in c16]
    p, q = plain[5], c16[5]
    assert (q.api_dtype, p.api_dtype) == (4, 2)                               # the library's GEMM_BF16_C16 / GEMM_BF16
    assert p.algorithmic_bytes() - q.algorithmic_bytes() == 2 * p.m * p.n     # the result is half as large
    small = config_problems(5, dtype=DTYPE_BF16, c16=True)[3]
    A, B, C = type(small)("t", DTYPE_BF16, 8, 6, 4, c16=True).operands()
    assert C.buf.dtype.itemsize == 2 and A.buf.dtype.itemsize == 2
    layer = conv_layer_problems("vgg16", dtype=DTYPE_BF16, c16=True)[8]
    assert layer.api_dtype == 4 and layer.name.endswith("_c16")
    assert layer.algorithmic_bytes() < conv_layer_problems("vgg16", dtype=DTYPE_BF16)[8].algorithmic_bytes()
