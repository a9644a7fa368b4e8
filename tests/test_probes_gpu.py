"""The library's own peak probes (Section IV-A's "solo mode" carried over to the three units that bound the kernels):
they run, return plausible rates for a B200, reject bad arguments and leave the device status clean."""
import pytest
import torch

import paper_2310_17408_b200 as g

pytestmark = pytest.mark.gpu


def stream():
    return torch.cuda.current_stream().cuda_stream


def test_copy_probe_moves_the_bytes_and_reports_a_rate():
    n = 256 << 20
    src = torch.arange(n // 8, dtype=torch.int64, device="cuda")
    dst = torch.zeros(n // 8, dtype=torch.int64, device="cuda")
    rc, gbs, ms = g.gemm_probe_copy(dst.data_ptr(), src.data_ptr(), n, stream())
    assert rc == 0
    assert torch.equal(src, dst)                      # bit-exact copy
    assert 1000.0 < gbs < 9000.0 and ms > 0.0
    assert abs(gbs - 2 * n / (ms * 1e-3) / 1e9) < 1e-6 * gbs      # rate = (read + written) / time
    # unaligned size, overlapping or unaligned pointers are refused
    assert g.gemm_probe_copy(dst.data_ptr(), src.data_ptr(), n + 8, stream())[0] < 0
    assert g.gemm_probe_copy(dst.data_ptr() + 8, src.data_ptr(), 1 << 20, stream())[0] < 0


@pytest.mark.parametrize("pattern,low,high", [(0, 40.0, 80.0), (1, 30.0, 80.0), (2, 30.0, 80.0)])
def test_ffma_probe_rates_are_below_the_alu_peak(pattern, low, high):
    rc, tf, ms = g.gemm_probe_ffma(pattern, 2048, stream())
    assert rc == 0
    assert low < tf < high and ms > 0.0               # 148 SMs x 128 lanes x 2 x 1.965 GHz = 74.4 TFLOP/s
    assert g.gemm_probe_ffma(3, 16, stream())[0] == -1
    assert g.gemm_probe_ffma(0, 0, stream())[0] == -2
    assert g.gemm_probe_ffma(0, (1 << 16) + 1, stream())[0] == -2


@pytest.mark.parametrize("dtype,pair", [(g.GEMM_BF16, 0), (g.GEMM_BF16, 1), (g.GEMM_F16, 1)])
def test_umma_probe_runs_on_every_sm_and_leaves_the_status_clean(dtype, pair):
    rc, tf, ms = g.gemm_probe_umma(dtype, pair, 20000, stream())
    assert rc == 0
    assert 500.0 < tf < 2600.0 and ms > 0.0           # nominal dense bf16 / f16 peak: 2250 TFLOP/s
    assert g.gemm_poll_status() == 0                  # no bounded wait expired
    assert g.gemm_probe_umma(g.GEMM_F32, 0, 100, stream())[0] < 0
    assert g.gemm_probe_umma(dtype, 2, 100, stream())[0] < 0
    assert g.gemm_probe_umma(dtype, pair, 0, stream())[0] < 0
