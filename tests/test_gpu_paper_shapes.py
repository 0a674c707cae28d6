"""GPU parity on the shapes the paper itself prints (its Gemmini GEMM listing, the schedule-reuse table, the
ablation's convolution, and int8 stand-ins for its Trainium GEMM / conv2d shapes), bit-exact against the oracle."""
import numpy as np
import pytest

from paper_2505_18574_b200 import inputs
import harness as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("i", range(len(inputs.SWEEP_GEMMS)), ids=lambda i: "x".join(map(str, inputs.SWEEP_GEMMS[i])))
def test_paper_gemm_shapes(i):
    import paper_2505_18574_b200 as i8
    p = inputs.sweep_gemm(i)
    i8.set_path(0)
    got = H.gemm_gpu(p)
    assert i8.last_path() in (i8.PATH_TENSOR, i8.PATH_TENSOR_2SM)
    if p.M * p.N * p.K <= 2 ** 36:
        want = H.gemm_oracle(p)
        H.assert_same(got, want, p.name)
    else:                                   # 4096 x 8192 x 8192: 512 sampled rows, every column
        rng = np.random.default_rng(i)
        rows = np.unique(np.concatenate([rng.integers(0, p.M, size=500), [0, 127, 128, p.M - 1]]))
        want = H.gemm_oracle_rows(p, rows)
        H.assert_same(got[rows], want, p.name)
    H.not_degenerate(want)


@pytest.mark.parametrize("i", range(len(inputs.SWEEP_CONVS)))
def test_paper_conv_shapes(i):
    import paper_2505_18574_b200 as i8
    p = inputs.sweep_conv(i)
    i8.set_path(0)
    got = H.conv_gpu(p)
    assert i8.last_path() in (i8.PATH_TENSOR, i8.PATH_TENSOR_2SM)
    if p.N * p.P * p.Q * p.K * p.R * p.S * p.C <= 2 ** 34:
        want = H.conv_oracle(p)
        H.assert_same(got, want, p.name)
    else:                                   # batch 16, 128x128x128 -> 512: the first and last image
        want0 = H.conv_oracle(p, 0, 1)
        want1 = H.conv_oracle(p, p.N - 1, p.N)
        H.assert_same(got[0], want0[0], p.name + " image 0")
        H.assert_same(got[-1], want1[-1], p.name + " last image")
        want = want0[0]
    H.not_degenerate(want)
