"""GPU parity on the shapes the paper itself prints (its Gemmini GEMM listing, the schedule-reuse table, the
ablation's convolution, and int8 stand-ins for its Trainium GEMM / conv2d shapes), bit-exact against the oracle."""
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
    assert i8.last_path() in (i8.PATH_TENSOR, i8.PATH_TENSOR_2SM, i8.PATH_CHANNEL_MAJOR, i8.PATH_CHANNEL_MAJOR_2SM)
    want = H.gemm_oracle(p)              # every element, also for 4096 x 8192 x 8192 (seconds of plain loops on the host)
    H.assert_same(got, want, p.name)
    H.not_degenerate(want)


@pytest.mark.parametrize("i", range(len(inputs.SWEEP_CONVS)))
def test_paper_conv_shapes(i):
    import paper_2505_18574_b200 as i8
    p = inputs.sweep_conv(i)
    i8.set_path(0)
    got = H.conv_gpu(p)
    assert i8.last_path() in (i8.PATH_TENSOR, i8.PATH_TENSOR_2SM, i8.PATH_CHANNEL_MAJOR, i8.PATH_CHANNEL_MAJOR_2SM)
    want = H.conv_oracle(p)              # every element, also for the batch-16 128x128x128 -> 512 layer
    H.assert_same(got, want, p.name)
    H.not_degenerate(want)
