"""Property tests on the GPU: random small shapes, paddings, scales and flags, each bit-exact against the oracle,
on the tensor path when the layout allows it and on the generic kernel otherwise."""
import numpy as np
import pytest
from hypothesis import HealthCheck, given, settings, strategies as st

from paper_2505_18574_b200 import inputs
import harness as H

pytestmark = pytest.mark.gpu

scales = st.one_of(
    st.tuples(st.integers(1 << 14, (1 << 15) - 1), st.integers(10, 24)),            # benchmark-like
    st.tuples(st.integers(-(1 << 31), (1 << 31) - 1), st.integers(0, 31)),            # anything legal
    st.sampled_from([(1, 0), (-1, 0), (0, 3), (-(1 << 31), 0), ((1 << 31) - 1, 31), (1, 31), (3, 1), (-(1 << 30), 31)]),
)


@settings(max_examples=40, deadline=None, suppress_health_check=list(HealthCheck))
@given(M=st.integers(1, 300), N=st.integers(1, 300), K16=st.integers(1, 24), seed=st.integers(0, 10 ** 6),
       pads=st.tuples(st.sampled_from([0, 16, 48]), st.sampled_from([0, 16, 32]), st.integers(0, 20)),
       relu=st.booleans(), per_channel=st.booleans(), with_bias=st.booleans(), scale=scales)
def test_random_gemms(M, N, K16, seed, pads, relu, per_channel, with_bias, scale):
    import paper_2505_18574_b200 as i8
    K = 16 * K16
    p = inputs.make_gemm(M, N, K, seed, per_channel=int(per_channel), relu=int(relu), with_bias=with_bias,
                         lda_pad=pads[0], ldb_pad=pads[1], ldc_pad=pads[2], shift_lo=8, shift_hi=20)
    if not per_channel:
        p.mult[:] = scale[0]; p.shift[:] = scale[1]
    else:
        p.mult[0] = scale[0]; p.shift[0] = scale[1]         # one channel with the drawn (possibly extreme) scale
    want = H.gemm_oracle(p)
    i8.set_path(0)
    got = H.gemm_gpu(p)
    assert i8.last_path() == i8.PATH_TENSOR
    H.assert_same(got, want, f"{p.name} seed {seed} tensor")
    i8.set_path(2)                                      # the same problem on the two-SM kernel
    got = H.gemm_gpu(p)
    assert i8.last_path() == i8.PATH_TENSOR_2SM
    i8.set_path(0)
    H.assert_same(got, want, f"{p.name} seed {seed} two-SM")


@settings(max_examples=15, deadline=None, suppress_health_check=list(HealthCheck))
@given(N=st.integers(1, 3), H_=st.integers(5, 40), W=st.integers(5, 40), C32=st.integers(1, 6), K=st.integers(1, 100),
       R=st.sampled_from([1, 3, 5]), stride=st.integers(1, 3), pad=st.integers(0, 2), seed=st.integers(0, 10 ** 6),
       relu=st.booleans())
def test_random_convs(N, H_, W, C32, K, R, stride, pad, seed, relu):
    import paper_2505_18574_b200 as i8
    if H_ + 2 * pad < R or W + 2 * pad < R:
        return
    C = 32 * C32
    batch = max(N, -(-131072 // (H_ * W * C)))          # large enough for the im2col tensor path
    p = inputs.make_conv(batch, H_, W, C, K, R, R, stride, pad, seed, relu=int(relu))
    want = H.conv_oracle(p)
    i8.set_path(0)
    got = H.conv_gpu(p)
    path = i8.last_path()
    assert path in (i8.PATH_TENSOR, i8.PATH_CONV_SLAB, i8.PATH_CHANNEL_MAJOR, i8.PATH_CHANNEL_MAJOR_2SM)
    H.assert_same(got, want, f"{p.name} seed {seed} path {path}")
    if path != i8.PATH_TENSOR:                          # also the large-tile implicit-GEMM kernel
        i8.set_path(3)
        got = H.conv_gpu(p)
        assert i8.last_path() == i8.PATH_TENSOR
        i8.set_path(0)
        H.assert_same(got, want, f"{p.name} seed {seed} implicit GEMM")


@settings(max_examples=15, deadline=None, suppress_health_check=list(HealthCheck))
@given(batch=st.integers(1, 40), M=st.integers(1, 64), N16=st.integers(1, 4), K16=st.integers(1, 4), seed=st.integers(0, 10 ** 6),
       ppb=st.booleans(), relu=st.booleans(), scale=scales)
def test_random_batched(batch, M, N16, K16, seed, ppb, relu, scale):
    import paper_2505_18574_b200 as i8
    p = inputs.make_batched(batch, M, 16 * N16, 16 * K16, seed, per_problem_bias=ppb, relu=int(relu))
    p.mult[:] = scale[0]; p.shift[:] = scale[1]
    want = H.batched_oracle(p)
    i8.set_path(0)
    got = H.batched_gpu(p)
    assert i8.last_path() == i8.PATH_SMALL
    H.assert_same(got, want, f"{p.name} seed {seed}")
