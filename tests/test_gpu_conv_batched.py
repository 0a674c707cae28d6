"""GPU parity: conv2d_i8 and batched_gemm_i8 through the C ABI against the CPU oracle, bit-exact."""
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


def _conv_both(p, expect_tensor=None):
    import paper_2505_18574_b200 as i8
    want = H.conv_oracle(p)
    i8.set_path(0)
    got = H.conv_gpu(p)
    path = i8.last_path()
    H.assert_same(got, want, f"{p.name} auto path={path}")
    if expect_tensor is not None:
        assert (path in (i8.PATH_TENSOR, i8.PATH_TENSOR_2SM, i8.PATH_CONV_SLAB, i8.PATH_CHANNEL_MAJOR, i8.PATH_CHANNEL_MAJOR_2SM)) == expect_tensor, f"{p.name}: path {path}"
    if path in (i8.PATH_CONV_SLAB, i8.PATH_CHANNEL_MAJOR, i8.PATH_CHANNEL_MAJOR_2SM):
        i8.set_path(3)                                   # the same layer on the large-tile implicit-GEMM kernel
        got = H.conv_gpu(p)
        assert i8.last_path() in (i8.PATH_TENSOR, i8.PATH_TENSOR_2SM, i8.PATH_GENERIC), f"{p.name}: path {i8.last_path()}"
        H.assert_same(got, want, f"{p.name} implicit GEMM (or generic, for small activations)")
    i8.set_path(1)
    got = H.conv_gpu(p)
    assert i8.last_path() == i8.PATH_GENERIC
    H.assert_same(got, want, f"{p.name} generic")
    return want


@pytest.mark.parametrize("N,H_,W,C,K,R,S,st,pad", [
    (1, 8, 8, 64, 64, 3, 3, 1, 1), (2, 9, 7, 64, 32, 3, 3, 1, 1), (3, 12, 12, 128, 64, 3, 3, 2, 1),
    (2, 7, 7, 256, 128, 1, 1, 1, 0), (1, 5, 5, 3, 4, 3, 3, 1, 1), (2, 10, 11, 16, 24, 5, 5, 2, 2),
    (2, 14, 14, 64, 96, 3, 3, 1, 0), (1, 6, 6, 32, 16, 1, 1, 2, 0), (4, 28, 28, 64, 64, 3, 3, 1, 1),
    (2, 15, 13, 192, 80, 3, 3, 2, 1), (1, 4, 4, 512, 64, 3, 3, 1, 1),
])
def test_conv_shapes(N, H_, W, C, K, R, S, st, pad):
    p = inputs.make_conv(N, H_, W, C, K, R, S, st, pad, 300 + N + H_ + C + K)
    _conv_both(p)


@pytest.mark.parametrize("N,H_,W,C,K,R,S,st,pad", [
    (4, 28, 28, 64, 64, 3, 3, 1, 1),      # 64-byte channel block, two taps per ring slot, odd tap count
    (8, 12, 12, 128, 64, 3, 3, 2, 1),     # 128-byte channel block, stride 2
    (4, 15, 13, 192, 80, 3, 3, 2, 1),     # 64-byte blocks x3, odd image, ragged filter count
    (8, 24, 24, 32, 48, 3, 3, 1, 1),      # 32-byte channel block, four taps per slot
    (4, 20, 22, 96, 40, 5, 5, 2, 2),      # 5x5 filter, 32-byte blocks x3
    (6, 14, 14, 256, 256, 3, 3, 1, 1),    # two 128-byte blocks per tap
    (5, 17, 17, 128, 136, 3, 3, 1, 0),    # no padding: the output is smaller than the input
    (9, 16, 16, 64, 64, 1, 1, 2, 0),      # strided 1x1
    (2, 40, 36, 64, 192, 3, 3, 1, 1),     # tiles spanning several rows and both images
    (3, 30, 30, 64, 64, 7, 7, 2, 3),      # 7x7 stride 2 pad 3
])
def test_conv_tensor_path(N, H_, W, C, K, R, S, st, pad):
    assert N * H_ * W * C >= 131072
    p = inputs.make_conv(N, H_, W, C, K, R, S, st, pad, 500 + N + H_ + C + K)
    _conv_both(p, expect_tensor=True)


@pytest.mark.parametrize("N,H_,W,C,K,R,S,st,pad", [
    (4, 28, 28, 64, 64, 3, 3, 1, 1), (8, 12, 12, 128, 64, 3, 3, 2, 1), (4, 15, 13, 192, 80, 3, 3, 2, 1), (8, 24, 24, 32, 48, 3, 3, 1, 1),
    (6, 14, 14, 256, 256, 3, 3, 1, 1), (5, 17, 17, 128, 136, 3, 3, 1, 0), (2, 40, 36, 64, 192, 3, 3, 1, 1), (3, 30, 30, 64, 64, 7, 7, 2, 3),
])
def test_conv_cta_pair_kernel(N, H_, W, C, K, R, S, st, pad):
    """The same convolutions forced onto clusters of two CTAs (cta_group::2, im2col loads counted on the even CTA)."""
    import paper_2505_18574_b200 as i8
    p = inputs.make_conv(N, H_, W, C, K, R, S, st, pad, 900 + N + H_ + C + K)
    want = H.conv_oracle(p)
    i8.set_path(2)
    got = H.conv_gpu(p)
    assert i8.last_path() == i8.PATH_TENSOR_2SM
    H.assert_same(got, want, p.name + " two-SM")


@pytest.mark.parametrize("N,H_,W,C,K,R,S,st,pad", [
    (1, 7, 7, 512, 512, 3, 3, 1, 1),      # the last ResNet-50 stage at batch 1: 25 KB of activations
    (1, 14, 14, 256, 256, 3, 3, 2, 1),    # stride 2, 50 KB
    (2, 9, 9, 48, 40, 5, 5, 3, 2),        # channels a multiple of 16 only, ragged filter count
    (1, 28, 28, 128, 160, 3, 3, 1, 0),    # 100 KB, no padding, several row tiles, too many filters for the slab kernel
    (4, 40, 40, 32, 64, 3, 3, 9, 1),      # a stride beyond the im2col loads' range on a large tensor
    (1, 20, 21, 16, 32, 17, 3, 1, 8),     # a filter side beyond the im2col loads' range
    (3, 5, 6, 16, 8, 2, 4, 1, 3),         # tiny: padding wider than the image's half
])
def test_conv_unfolded_layers_take_the_tensor_path(N, H_, W, C, K, R, S, st, pad):
    """Layers outside the im2col loads' reach (small activation tensors, long strides, large filters) with C % 16 == 0:
    unfold pass + tensor GEMM, bit-exact against the oracle; the generic kernel when the unfold path is ruled out."""
    import paper_2505_18574_b200 as i8
    p = inputs.make_conv(N, H_, W, C, K, R, S, st, pad, 1300 + N + H_ + C + K)
    want = H.conv_oracle(p)
    got = H.conv_gpu(p)
    assert i8.last_conv_unfolded(), p.name
    assert i8.last_path() in (i8.PATH_TENSOR, i8.PATH_TENSOR_2SM, i8.PATH_CHANNEL_MAJOR, i8.PATH_CHANNEL_MAJOR_2SM), i8.last_path()
    H.assert_same(got, want, p.name + " unfolded")
    H.assert_same(H.conv_gpu(p), want, p.name + " unfolded, second call (workspace reused from the pool)")
    i8.set_path(1)
    H.assert_same(H.conv_gpu(p), want, p.name + " generic")
    assert not i8.last_conv_unfolded() and i8.last_path() == i8.PATH_GENERIC


@pytest.mark.parametrize("N,H_,W,C,K,R,S,st,pad", [
    (4, 32, 32, 3, 64, 7, 7, 2, 3),       # an RGB first layer: 147 columns padded to 160
    (2, 15, 17, 20, 24, 3, 3, 1, 1),      # channels a multiple of 4 only
    (3, 9, 9, 7, 5, 2, 2, 1, 0),          # odd everything
    (16, 56, 56, 8, 32, 3, 3, 1, 1),      # a large activation tensor with 8 channels
])
def test_conv_with_any_channel_count_takes_the_tensor_path(N, H_, W, C, K, R, S, st, pad):
    """Channel counts that are not a multiple of 16: byte-wise unfold, padded copy of the filters, tensor GEMM."""
    import paper_2505_18574_b200 as i8
    p = inputs.make_conv(N, H_, W, C, K, R, S, st, pad, 1500 + N + H_ + C + K)
    want = H.conv_oracle(p)
    got = H.conv_gpu(p)
    assert i8.last_conv_unfolded() and i8.last_path() in (i8.PATH_TENSOR, i8.PATH_TENSOR_2SM, i8.PATH_CHANNEL_MAJOR, i8.PATH_CHANNEL_MAJOR_2SM), i8.last_path()
    H.assert_same(got, want, p.name + " unfolded byte-wise")
    i8.set_path(1)
    H.assert_same(H.conv_gpu(p), want, p.name + " generic")
    assert not i8.last_conv_unfolded()


def test_conv_unfolded_inside_a_cuda_graph_and_on_two_streams():
    """The unfold workspace lives in stream order: a captured graph owns its copy (replays give the same bytes), and two
    streams running different layers at once do not share it."""
    import torch
    import paper_2505_18574_b200 as i8
    dev = torch.device("cuda", 0)
    ps = [inputs.make_conv(1, 14, 14, 256, 256, 3, 3, 1, 1, 1401), inputs.make_conv(1, 7, 7, 512, 384, 3, 3, 1, 1, 1402)]
    wants = [H.conv_oracle(p) for p in ps]

    def dev_args(p):
        T = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        y = torch.zeros((p.N, p.P, p.Q, p.K), dtype=torch.int8, device=dev)
        return (T(p.x), T(p.w), y, T(p.bias), T(p.mult), T(p.shift), p.per_channel, p.relu, (p.stride_h, p.stride_w), (p.pad_h, p.pad_w))

    args = [dev_args(p) for p in ps]
    # two streams, interleaved launches
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for _ in range(8):
        for a, s in zip(args, streams):
            with torch.cuda.stream(s):
                i8.conv2d_i8(*a)
                assert i8.last_conv_unfolded()
    torch.cuda.synchronize()
    for a, w, p in zip(args, wants, ps):
        H.assert_same(a[2].cpu().numpy(), w, p.name + " two streams")
        a[2].zero_()
    # graph capture and three replays
    g = torch.cuda.CUDAGraph(); s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            for a in args:
                i8.conv2d_i8(*a)
    for _ in range(3):
        for a in args:
            a[2].zero_()
        g.replay(); torch.cuda.synchronize()
        for a, w, p in zip(args, wants, ps):
            H.assert_same(a[2].cpu().numpy(), w, p.name + " graph replay")
    assert i8.last_device_status() == 0


def test_conv_delta_filter_on_gpu():
    """Oracle-independent: a filter with a single 1 copies a shifted view of the input."""
    import paper_2505_18574_b200 as i8
    p = inputs.make_conv(24, 9, 10, 64, 64, 3, 3, 1, 1, 5, per_channel=0, relu=0, with_bias=False, act_lo=-100, act_hi=101)
    p.mult[:] = 1; p.shift[:] = 0
    for (r, s, mode) in [(0, 0, 0), (1, 1, 0), (2, 0, 0), (1, 2, 0), (0, 2, 3), (2, 1, 3)]:
        p.w[:] = 0
        for k in range(64):
            p.w[k, r, s, (k + 3) % 64] = 1
        i8.set_path(mode)
        got = H.conv_gpu(p)
        assert i8.last_path() == (i8.PATH_CONV_SLAB if mode == 0 else i8.PATH_TENSOR)
        for pp in range(p.P):
            for q in range(p.Q):
                h = pp - 1 + r; w = q - 1 + s
                want = p.x[:, h, w, :][:, [(k + 3) % 64 for k in range(64)]] if (0 <= h < 9 and 0 <= w < 10) else 0
                assert np.array_equal(got[:, pp, q, :], np.broadcast_to(want, (24, 64))), (r, s, pp, q)


@pytest.mark.parametrize("N,H_,W,C,K,R,S,pad", [
    (3, 56, 56, 64, 64, 3, 3, (1, 1)),      # the 56 x 56 x 64 layer: two output rows per tile, 64-byte channel block
    (5, 14, 14, 128, 128, 3, 3, (1, 1)),    # eight rows per tile, 128-byte channel block, 128 filters
    (3, 14, 14, 256, 48, 3, 3, (1, 1)),     # two 128-byte channel blocks per tile
    (4, 27, 31, 32, 40, 3, 3, (1, 1)),      # 32-byte block, ragged filter count, odd extents (row count not a multiple of the tile)
    (2, 20, 100, 64, 64, 3, 3, (1, 1)),     # one row per tile (raster width 102)
    (3, 19, 23, 96, 40, 5, 5, (2, 2)),      # 5 x 5 filter, three 32-byte blocks
    (2, 33, 40, 64, 24, 3, 3, (0, 0)),      # no padding: output smaller than the input
    (2, 30, 30, 32, 64, 7, 7, (3, 3)),      # 7 x 7 filter
    (3, 18, 25, 128, 64, 3, 5, (1, 2)),     # rectangular filter with matching padding
    (2, 24, 24, 64, 64, 3, 3, (2, 0)),      # unequal padding: taller output, narrower output
    (1, 9, 62, 96, 8, 1, 3, (0, 1)),        # 1 x 3 filter, 8 filters
    (7, 12, 12, 64, 64, 3, 3, (1, 1)),      # nine of the twelve rows in one tile, three in the next
    (40, 28, 28, 64, 64, 3, 3, (1, 1)),     # 280 tiles: both issuers of every CTA take a turn
])
def test_conv_slab_kernel(N, H_, W, C, K, R, S, pad):
    """Stride-1 layers with few filters run on the slab kernel (input rows resident in shared memory, taps read
    through row-shifted descriptors); same results as the oracle and as the library's other kernels."""
    import paper_2505_18574_b200 as i8
    p = inputs.make_conv(N, H_, W, C, K, R, S, 1, 0, 700 + N + H_ + C + K)
    p.pad_h, p.pad_w = pad
    want = H.conv_oracle(p)
    assert want.shape == (N, H_ + 2 * pad[0] - R + 1, W + 2 * pad[1] - S + 1, K)
    i8.set_path(0)
    got = H.conv_gpu(p)
    assert i8.last_path() == i8.PATH_CONV_SLAB, f"{p.name}: path {i8.last_path()}"
    H.assert_same(got, want, p.name + " slab")
    assert len(np.unique(want)) > 32, "degenerate output would prove nothing"
    i8.set_path(3)
    got = H.conv_gpu(p)
    assert i8.last_path() != i8.PATH_CONV_SLAB
    H.assert_same(got, want, p.name + " without the slab kernel")
    assert i8.last_device_status() == 0


@pytest.mark.parametrize("seed", range(16))
def test_seeded_random_stride1_convs(seed):
    """Random stride-1 layers up to the slab kernel's limits (raster width 128, 128 filters, filter bank in shared memory):
    whichever kernel the dispatcher picks must agree with the oracle, and so must the implicit-GEMM / generic choice."""
    import paper_2505_18574_b200 as i8
    rng = np.random.default_rng(4000 + seed)
    R = int(rng.choice([1, 3, 5])); S = int(rng.choice([1, 3, 5]))
    ph = int(rng.integers(0, R // 2 + 1)); pw = int(rng.integers(0, S // 2 + 1))
    W = int(rng.choice([S, 7, 14, 28, 56, 100, 124, 126, 128 - 2 * pw, 130]))
    H_ = int(rng.integers(R, 30)); N = int(rng.integers(1, 5))
    C = int(rng.choice([32, 64, 96, 128])); K = int(rng.choice([1, 8, 40, 64, 65, 100, 128, 136]))
    if R == 1 and S == 1:
        ph = pw = 1                                       # keep it off the 1x1 -> GEMM shortcut
    p = inputs.make_conv(N, H_, W, C, K, R, S, 1, 0, 4100 + seed, relu=int(rng.integers(0, 2)))
    p.pad_h, p.pad_w = ph, pw
    want = H.conv_oracle(p)
    paths = []
    for mode in (0, 3):
        i8.set_path(mode)
        got = H.conv_gpu(p)
        paths.append(i8.last_path())
        H.assert_same(got, want, f"{p.name} pad ({ph},{pw}) seed {seed} mode {mode} path {paths[-1]}")
    i8.set_path(0)
    assert paths[1] != i8.PATH_CONV_SLAB
    assert i8.last_device_status() == 0


def test_conv_1x1_equals_gemm_on_gpu():
    p = inputs.make_conv(3, 7, 7, 128, 256, 1, 1, 1, 0, 8)
    y = H.conv_gpu(p)
    g = inputs.make_gemm(3 * 49, 256, 128, 0, per_channel=1, relu=1)
    g.A = p.x.reshape(-1, 128).copy(); g.B = p.w.reshape(256, 128).copy()
    g.bias, g.mult, g.shift = p.bias, p.mult, p.shift
    H.assert_same(y.reshape(-1, 256), H.gemm_gpu(g), "1x1 conv vs gemm")


def test_config2_conv():
    p = inputs.config2()
    want = H.conv_oracle(p)
    H.assert_same(H.conv_gpu(p), want, p.name)
    H.not_degenerate(want)


@pytest.mark.parametrize("j", [0, 1, 2])
def test_config3_conv_mix(j):
    p = inputs.config3(j)
    want = H.conv_oracle(p)
    H.assert_same(H.conv_gpu(p), want, p.name)
    H.not_degenerate(want)


@pytest.mark.parametrize("batch,M,N,K,ppb", [(1, 64, 64, 64, True), (7, 64, 64, 64, True), (8, 64, 64, 64, False),
                                             (5, 32, 48, 80, True), (3, 128, 64, 64, True), (9, 17, 19, 23, True),
                                             (33, 64, 64, 64, True)])
def test_batched_shapes(batch, M, N, K, ppb):
    import paper_2505_18574_b200 as i8
    p = inputs.make_batched(batch, M, N, K, 400 + batch + M, per_problem_bias=ppb)
    p.shift[:] = 14
    want = H.batched_oracle(p)
    for mode in (0, 1):
        i8.set_path(mode)
        H.assert_same(H.batched_gpu(p), want, f"{p.name} mode {mode}")
        if mode == 0 and M % 16 == 0 and N % 16 == 0 and K % 16 == 0:
            assert i8.last_path() != i8.PATH_GENERIC, "aligned problems run on a tensor path, whatever their size"


@pytest.mark.parametrize("batch,M,N,K", [(3, 128, 128, 128), (5, 256, 192, 320), (2, 130, 144, 80), (40, 128, 128, 128), (4, 1024, 512, 256)])
def test_batched_problems_larger_than_the_paired_tile(batch, M, N, K):
    """Problems above 64 in any dimension on the large-tile kernel (row-major B through the MN-major descriptor), per-problem
    bias."""
    import paper_2505_18574_b200 as i8
    p = inputs.make_batched(batch, M, N, K, 700 + batch + M + N)
    p.shift[:] = 24
    want = H.batched_oracle(p)
    i8.set_path(0)
    got = H.batched_gpu(p)
    assert i8.last_path() in (i8.PATH_TENSOR, i8.PATH_TENSOR_2SM, i8.PATH_CHANNEL_MAJOR, i8.PATH_CHANNEL_MAJOR_2SM), i8.last_path()
    H.assert_same(got, want, p.name)
    H.not_degenerate(want)


@pytest.mark.parametrize("batch,M,N,K,ppb", [(6, 200, 144, 96, True), (300, 96, 80, 112, True), (17, 128, 304, 272, False),
                                             (64, 128, 128, 128, True), (9, 65, 16, 1040, True)])
@pytest.mark.parametrize("b_col_major", [False, True])
def test_batched_problems_in_one_launch(batch, M, N, K, ppb, b_col_major):
    """Problems above the paired 64^3 tile, all in one launch of the large-tile kernel: the tile schedule runs over the
    stacked problems (block rows of A that cross into the next problem are never stored), either storage order of B,
    per-problem and shared bias, a padded batch stride of C whose gaps must stay untouched."""
    import torch
    import paper_2505_18574_b200 as i8
    p = inputs.make_batched(batch, M, N, K, 800 + batch + M + N + K, per_problem_bias=ppb)
    p.shift[:] = 22
    want = H.batched_oracle(p)
    A = torch.from_numpy(p.A).cuda()
    if b_col_major:
        B = torch.from_numpy(np.ascontiguousarray(p.B.transpose(0, 2, 1))).cuda().transpose(1, 2)   # (batch, K, N) view, K contiguous
    else:
        B = torch.from_numpy(p.B).cuda()
    Cbuf = torch.full((batch, M + 3, N), 0x5A, dtype=torch.int8, device="cuda")                      # three spare rows per problem
    C = Cbuf[:, :M, :]
    bias, mult, shift = (torch.from_numpy(v).cuda() for v in (p.bias, p.mult, p.shift))
    for mode in (0, 1):
        i8.set_path(mode)
        Cbuf.fill_(0x5A)
        i8.batched_gemm_i8(A, B, C, bias, mult, shift, p.per_channel, p.relu)
        assert i8.last_device_status() == 0
        assert (i8.last_path() == i8.PATH_TENSOR) if mode == 0 else (i8.last_path() == i8.PATH_GENERIC), i8.last_path()
        H.assert_same(C.cpu().numpy(), want, f"{p.name} mode {mode} b_col_major={b_col_major}")
        assert (Cbuf[:, M:, :] == 0x5A).all(), "rows between the problems of C were written"
    if batch > 8:
        plan = i8.last_plan()        # generic mode ran last: the plan still shows the tensor launch before it
        assert plan["m_tiles"] == batch * ((M + 127) // 128), plan
    i8.set_path(0)
    H.not_degenerate(want)


@pytest.mark.parametrize("batch,M,N,K", [(2, 64, 64, 64), (7, 64, 64, 64), (1, 64, 64, 64), (6, 64, 32, 64), (5, 17, 64, 48),
                                         (4, 64, 16, 16), (9, 40, 48, 32), (300, 64, 64, 64), (3, 1, 64, 64)])
@pytest.mark.parametrize("b_col_major", [False, True])
def test_batched_small_tile_path(batch, M, N, K, b_col_major):
    """Paired small-tile kernel: row-major B goes through an MN-major descriptor, column-major B through a K-major one."""
    import torch
    import paper_2505_18574_b200 as i8
    p = inputs.make_batched(batch, M, N, K, 600 + batch + M + N + K)
    p.shift[:] = 13
    want = H.batched_oracle(p)
    A = torch.from_numpy(p.A).cuda()
    if b_col_major:
        B = torch.from_numpy(np.ascontiguousarray(p.B.transpose(0, 2, 1))).cuda().transpose(1, 2)   # (batch, K, N) view, K contiguous
    else:
        B = torch.from_numpy(p.B).cuda()
    C = torch.full((batch, M, N), 0x5A, dtype=torch.int8, device="cuda")
    i8.set_path(0)
    i8.batched_gemm_i8(A, B, C, torch.from_numpy(p.bias).cuda(), torch.from_numpy(p.mult).cuda(), torch.from_numpy(p.shift).cuda(),
                       p.per_channel, p.relu)
    assert i8.last_device_status() == 0
    assert i8.last_path() == i8.PATH_SMALL
    H.assert_same(C.cpu().numpy(), want, f"{p.name} b_col_major={b_col_major}")


@pytest.mark.parametrize("mult,shift,relu,per_channel", [(1, 0, 0, 0), (-3, 1, 1, 0), (2147483647, 31, 0, 0), (20000, 20, 1, 1), (0, 7, 0, 0)])
def test_batched_small_tile_scales(mult, shift, relu, per_channel):
    import paper_2505_18574_b200 as i8
    p = inputs.make_batched(5, 64, 64, 64, 9, relu=relu)
    if per_channel:
        rng = np.random.default_rng(4)
        p.mult = rng.integers(-(1 << 15), 1 << 15, size=64, dtype=np.int32)
        p.shift = rng.integers(0, 25, size=64, dtype=np.int32)
        p.per_channel = 1
    else:
        p.mult[:] = mult; p.shift[:] = shift
    want = H.batched_oracle(p)
    i8.set_path(0)
    got = H.batched_gpu(p)
    assert i8.last_path() == i8.PATH_SMALL
    H.assert_same(got, want, p.name)


def test_config4b_batched():
    import paper_2505_18574_b200 as i8
    p = inputs.config4b()
    want = H.batched_oracle(p)
    H.assert_same(H.batched_gpu(p), want, p.name)
    assert i8.last_path() == i8.PATH_SMALL
    H.not_degenerate(want)
