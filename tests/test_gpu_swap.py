"""GPU parity of the channel-major tensor kernel (output channels on the tensor-memory lanes, a strip of output rows on
the columns): forced with path mode 4 and compared element by element with the CPU oracle, for GEMMs and convolutions, on
one CTA per tile (at most 128 channels) and on CTA pairs."""
import numpy as np
import pytest

from paper_2505_18574_b200 import inputs
import harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _auto_path():
    import paper_2505_18574_b200 as i8
    i8.set_path(0)
    yield
    i8.set_path(0)


def _swap_paths():
    import paper_2505_18574_b200 as i8
    return (i8.PATH_CHANNEL_MAJOR, i8.PATH_CHANNEL_MAJOR_2SM)


@pytest.mark.parametrize("M,N,K", [
    (128, 128, 128), (256, 256, 128), (16, 128, 32), (1, 16, 16), (127, 65, 129), (129, 257, 33), (300, 200, 100),
    (513, 96, 1040), (64, 700, 256), (1000, 40, 48), (5, 7, 16), (130, 130, 2048), (384, 320, 16), (128, 8, 64),
    (3136, 2048, 512), (12544, 256, 1152), (5000, 640, 256), (9001, 300, 64), (777, 1030, 272), (40000, 128, 64),
])
def test_gemm_shapes(M, N, K):
    """Ragged rows, channels and K; narrow and wide strips; one and several channel blocks."""
    import paper_2505_18574_b200 as i8
    pad = (-K) % 16
    for per_channel, relu in ((1, M % 2), (0, 1 - M % 2)):
        p = inputs.make_gemm(M, N, K, 6000 + M + N + K, per_channel=per_channel, relu=relu, shift_lo=12, shift_hi=22,
                             lda_pad=pad, ldb_pad=pad, ldc_pad=16 * per_channel)
        want = H.gemm_oracle(p)
        # 4: single CTAs or CTA pairs by the cost model; 5: pairs whenever there are more than 128 channels; 6: single CTAs
        for mode in (4, 5, 6):
            i8.set_path(mode)
            got = H.gemm_gpu(p)
            if mode == 4:
                assert i8.last_path() in _swap_paths(), i8.last_path()
            else:
                assert i8.last_path() == (i8.PATH_CHANNEL_MAJOR_2SM if N > 128 and mode == 5 else i8.PATH_CHANNEL_MAJOR), i8.last_path()
            H.assert_same(got, want, f"{p.name} mode {mode}")
    assert i8.last_device_status() == 0


@pytest.mark.parametrize("N,ldc_pad", [(13, 3), (200, 8), (135, 9), (1000, 24), (272, 16), (16, 0), (100, 5)])
def test_never_writes_outside_c(N, ldc_pad):
    """Channel counts that are not a multiple of 16 and padded or odd leading dimensions take the direct byte stores;
    the harness checks the padding columns and the guard bytes around C."""
    import paper_2505_18574_b200 as i8
    p = inputs.make_gemm(300, N, 64, 6100 + N, per_channel=1, relu=0, ldc_pad=ldc_pad, shift_lo=10, shift_hi=16)
    want = H.gemm_oracle(p)
    i8.set_path(4)
    H.assert_same(H.gemm_gpu(p), want, p.name)
    assert i8.last_path() in _swap_paths()


@pytest.mark.parametrize("mult,shift,relu", [(1, 0, 0), (-1, 0, 0), (2147483647, 31, 0), (-2147483648, 0, 0), (-2147483648, 31, 1),
                                              (0, 5, 0), (3, 1, 1), (65536, 16, 0), (-20000, 20, 1), (1, 31, 0),
                                              (1, 1, 0), (1, 2, 1), (-1, 2, 0), (3, 3, 0), (1048575, 21, 1), (-1048575, 21, 0),
                                              (1048576, 22, 0), (524287, 20, 0), (32767, 16, 1), (-3, 3, 0)])
def test_extreme_scales(mult, shift, relu):
    """Every epilogue form (folded, shift-32 with ReLU ahead of a negative multiplier, window) on per-thread constants."""
    import paper_2505_18574_b200 as i8
    p = inputs.make_gemm(160, 288, 64, 9, per_channel=1, relu=relu)
    p.mult[:] = mult; p.shift[:] = shift
    p.mult[::3] = 20000; p.shift[::3] = 22          # neighbouring channels (lanes of one warp) in different forms
    want = H.gemm_oracle(p)
    i8.set_path(4)
    H.assert_same(H.gemm_gpu(p), want, p.name)
    assert i8.last_path() in _swap_paths()


def test_closed_forms_on_gpu():
    """Oracle-independent: all-ones operands give K everywhere; a one-hot A row picks a row of B (no transposition or
    channel permutation survives this)."""
    import paper_2505_18574_b200 as i8
    i8.set_path(4)
    p = inputs.make_gemm(200, 384, 96, 3, per_channel=0, relu=0, with_bias=False)
    p.A[:] = 1; p.B[:] = 1; p.mult[:] = 1; p.shift[:] = 0
    got = H.gemm_gpu(p)
    assert i8.last_path() in _swap_paths() and (got == 96).all()
    p = inputs.make_gemm(96, 384, 96, 4, per_channel=0, relu=0, with_bias=False)
    p.A[:] = 0
    for i in range(96):
        p.A[i, (7 * i + 3) % 96] = 1
    p.mult[:] = 1; p.shift[:] = 0
    got = H.gemm_gpu(p)
    want = np.stack([p.B[:, (7 * i + 3) % 96] for i in range(96)])     # row i of C = column (7i+3)%96 of the (N, K) storage
    assert np.array_equal(got, want)


CONVS = [  # (N, H, W, C, K, R, S, stride, pad)
    (2, 12, 12, 64, 64, 3, 3, 1, 1), (3, 14, 14, 256, 256, 3, 3, 1, 1), (4, 28, 28, 128, 256, 3, 3, 2, 1),
    (2, 17, 13, 32, 160, 3, 3, 2, 1), (1, 9, 9, 96, 128, 5, 5, 1, 2), (5, 8, 8, 128, 300, 1, 1, 1, 0),
    (2, 20, 20, 64, 512, 3, 3, 1, 0), (64, 7, 7, 512, 2048, 1, 1, 1, 0), (8, 16, 16, 32, 48, 2, 2, 2, 0),
]


@pytest.mark.parametrize("shape", CONVS, ids=lambda s: "x".join(map(str, s)))
def test_conv_shapes(shape):
    import paper_2505_18574_b200 as i8
    N, Hh, W, C, K, R, S, st, pad = shape
    p = inputs.make_conv(N, Hh, W, C, K, R, S, st, pad, 6200 + sum(shape))
    want = H.conv_oracle(p)
    for mode in (4, 5, 6):
        i8.set_path(mode)
        got = H.conv_gpu(p)
        assert i8.last_path() in _swap_paths(), i8.last_path()      # small activation tensors: unfold pass + this kernel
        H.assert_same(got, want, f"{p.name} mode {mode}")
    assert i8.last_device_status() == 0


@pytest.mark.parametrize("j", [0, 1, 2])
def test_config3_conv_mix_channel_major(j):
    """The ResNet-like layer mix at full size on the channel-major kernel."""
    import paper_2505_18574_b200 as i8
    p = inputs.config3(j)
    want = H.conv_oracle(p)
    for mode in (5, 6):
        i8.set_path(mode)
        got = H.conv_gpu(p)
        assert i8.last_path() == (i8.PATH_CHANNEL_MAJOR_2SM if mode == 5 else i8.PATH_CHANNEL_MAJOR)
        H.assert_same(got, want, f"{p.name} mode {mode}")
    H.not_degenerate(want)


@pytest.mark.parametrize("M,N,K,per_channel,relu", [(300, 200, 112, 1, 0), (1000, 520, 272, 1, 1), (64, 40, 48, 0, 1), (2048, 256, 1024, 1, 0),
                                                    (129, 257, 33, 0, 0)])
def test_float_scale_readout(M, N, K, per_channel, relu):
    """gemm_i8_fscale (the scale as a binary32 float, round to nearest even) against its oracle, on the tensor path and on
    the generic kernel; scales with full mantissas so that both binary32 roundings matter."""
    import torch
    import oracle
    import paper_2505_18574_b200 as i8
    pad = (-K) % 16
    p = inputs.make_gemm(M, N, K, 6400 + M + N, per_channel=per_channel, relu=relu, lda_pad=pad, ldb_pad=pad)
    rng = np.random.default_rng(M + N)
    nq = N if per_channel else 1
    scale = (rng.uniform(0.5, 1.0, size=nq) * 2.0 ** rng.integers(-14, -8, size=nq)).astype(np.float32)
    scale[::5] *= -1.0
    want = oracle.gemm_i8_fscale(p.A, p.a_rs, 1, p.B, 1, p.b_cs, N, p.bias, scale, per_channel, M, N, K, relu)
    A = torch.from_numpy(p.A).cuda()[:, :K]; B = torch.from_numpy(p.B).cuda()[:, :K]
    bias = torch.from_numpy(p.bias).cuda(); sc = torch.from_numpy(scale).cuda()
    for mode in (0, 1, 5, 6):
        i8.set_path(mode)
        C = torch.full((M, N), 0x5A, dtype=torch.int8, device="cuda")
        i8.gemm_i8_fscale(A, B.t(), C, bias, sc, per_channel, relu)
        assert i8.last_device_status() == 0
        if mode == 0:
            assert i8.last_path() in _swap_paths()
        else:
            assert i8.last_path() == (i8.PATH_GENERIC if mode == 1 else (i8.PATH_CHANNEL_MAJOR_2SM if N > 128 and mode == 5 else i8.PATH_CHANNEL_MAJOR))
        H.assert_same(C.cpu().numpy(), want, f"float scale mode {mode}")
    H.not_degenerate(want)
    # large accumulators: |t| above 2^24 is rounded by the conversion itself
    p.A[:] = 127; p.B[:] = 127
    A = torch.from_numpy(p.A).cuda()[:, :K]; B = torch.from_numpy(p.B).cuda()[:, :K]
    big = np.full(nq, 1.0 / (127 * 127 * K) * 100.3, dtype=np.float32)
    want = oracle.gemm_i8_fscale(p.A, p.a_rs, 1, p.B, 1, p.b_cs, N, p.bias, big, per_channel, M, N, K, relu)
    i8.set_path(0)
    C = torch.empty((M, N), dtype=torch.int8, device="cuda")
    i8.gemm_i8_fscale(A, B.t(), C, bias, torch.from_numpy(big).cuda(), per_channel, relu)
    H.assert_same(C.cpu().numpy(), want, "float scale, constant operands")
