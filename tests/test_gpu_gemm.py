"""GPU parity: gemm_i8 through the C ABI against the CPU oracle, bit-exact."""
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


TENSOR_PATHS = (2, 4, 6, 7)      # large-tile kernel on one CTA / CTA pairs, channel-major kernel on one CTA / CTA pairs


def _both_paths(p, expect_tensor=True, two_sm=False):
    import paper_2505_18574_b200 as i8
    want = H.gemm_oracle(p)
    i8.set_path(2 if two_sm else 0)
    got = H.gemm_gpu(p)
    path = i8.last_path()
    H.assert_same(got, want, f"{p.name} auto path={path}")
    if two_sm:
        assert path == i8.PATH_TENSOR_2SM, f"{p.name}: expected the two-SM kernel, got {path}"
    elif expect_tensor:
        assert path in TENSOR_PATHS, f"{p.name}: expected a tensor path, got {path}"
    i8.set_path(1)
    got = H.gemm_gpu(p)
    assert i8.last_path() == i8.PATH_GENERIC
    H.assert_same(got, want, f"{p.name} generic")
    return want


@pytest.mark.parametrize("M,N,K,lda_pad,ldb_pad,a_off,b_off", [
    (200, 136, 100, 3, 5, 0, 0),         # leading dimensions that are not multiples of 16, ragged K
    (512, 384, 256, 0, 0, 1, 0),         # A starts one byte off a 16-byte boundary, B is fetched in place
    (300, 520, 272, 16, 0, 0, 7),        # B's base is off, A in place with a padded (still aligned) leading dimension
    (1000, 96, 33, 1, 1, 3, 5),          # everything off at once
    (4096, 1024, 512, 8, 8, 0, 0),       # large enough for 256-wide tiles
])
def test_operands_the_tensor_path_cannot_fetch_in_place_are_packed(M, N, K, lda_pad, ldb_pad, a_off, b_off):
    """Misaligned bases and leading dimensions: packed copies in the stream-ordered workspace, then a tensor kernel."""
    import torch
    import paper_2505_18574_b200 as i8
    p = inputs.make_gemm(M, N, K, 4700 + M + N + K, per_channel=1, relu=M % 2, shift_lo=19, shift_hi=25, lda_pad=lda_pad, ldb_pad=ldb_pad)
    want = H.gemm_oracle(p)
    lda, ldb = p.A.shape[1], p.B.shape[1]

    def shifted(host, off):
        flat = torch.zeros(host.size + 16 + off, dtype=torch.int8, device="cuda")
        base = (-flat.data_ptr()) % 16 + off                     # `off` bytes past a 16-byte boundary
        flat[base:base + host.size] = torch.from_numpy(host.reshape(-1)).cuda()
        return flat[base:base + host.size].view(host.shape)

    A = shifted(p.A, a_off)[:, :K]; B = shifted(p.B, b_off)[:, :K]
    assert A.data_ptr() % 16 == a_off and B.data_ptr() % 16 == b_off
    bias, mult, shift = (torch.from_numpy(v).cuda() for v in (p.bias, p.mult, p.shift))
    for mode in (0, 1):
        i8.set_path(mode)
        C = torch.full((M, N), 0x5A, dtype=torch.int8, device="cuda")
        i8.gemm_i8(A, B.t(), C, bias, mult, shift, p.per_channel, p.relu)
        assert i8.last_device_status() == 0
        if mode == 0:
            assert i8.last_gemm_packed() and i8.last_path() in TENSOR_PATHS, (i8.last_gemm_packed(), i8.last_path())
        else:
            assert not i8.last_gemm_packed() and i8.last_path() == i8.PATH_GENERIC
        H.assert_same(C.cpu().numpy(), want, f"{p.name} mode {mode} lda {lda} ldb {ldb}")
    i8.set_path(0)
    H.not_degenerate(want)


def test_config0_256cube():
    want = _both_paths(inputs.config0())
    H.not_degenerate(want)


def test_single_tile_structured():
    """Identity-like A and ramp B: a wrong descriptor field would show up as a recognisable permutation."""
    M = N = K = 128
    p = inputs.make_gemm(M, N, K, 1, per_channel=0, relu=0, with_bias=False)
    p.A[:] = 0
    for i in range(M):
        p.A[i, i] = 1
    for n in range(N):
        for k in range(K):
            p.B[n, k] = ((3 * k + 5 * n) % 251) - 125
    p.mult[:] = 1; p.shift[:] = 0
    want = _both_paths(p)
    assert np.array_equal(want, p.B.T[:K, :N])     # I . B = B, no scaling


@pytest.mark.parametrize("M,N,K", [
    (128, 128, 128), (128, 256, 128), (128, 64, 32), (256, 512, 384), (1, 16, 16), (127, 65, 129),
    (129, 257, 33), (300, 200, 100), (513, 96, 1040), (64, 700, 256), (1000, 40, 48), (5, 7, 16),
    (130, 130, 2048), (384, 320, 16), (128, 8, 64),
])
def test_ragged_shapes(M, N, K):
    # leading dimensions are padded to a multiple of 16 so the operands qualify for the tensor path
    pad = (-K) % 16
    p = inputs.make_gemm(M, N, K, 1000 + M + N + K, per_channel=1, relu=(M % 2), shift_lo=12, shift_hi=22,
                         lda_pad=pad, ldb_pad=pad)
    _both_paths(p)


@pytest.mark.parametrize("M,N,K,pads", [(200, 136, 96, (16, 32, 16)), (130, 70, 80, (48, 16, 3)), (64, 64, 64, (0, 0, 5))])
def test_padded_leading_dimensions(M, N, K, pads):
    p = inputs.make_gemm(M, N, K, 77, per_channel=1, relu=1, lda_pad=pads[0], ldb_pad=pads[1], ldc_pad=pads[2],
                         shift_lo=12, shift_hi=20)
    _both_paths(p)


@pytest.mark.parametrize("a_layout,b_layout", [("row", "row"), ("col", "col"), ("col", "row")])
def test_other_layouts_unaligned_use_generic(a_layout, b_layout):
    """Leading dimensions that are not multiples of 16 bytes cannot be described to the copy engine."""
    p = inputs.make_gemm(70, 50, 90, 5, a_layout=a_layout, b_layout=b_layout, per_channel=1, relu=0, shift_lo=10, shift_hi=18)
    _both_paths(p, expect_tensor=False)


@pytest.mark.parametrize("a_layout,b_layout", [("row", "row"), ("col", "col"), ("col", "row")])
@pytest.mark.parametrize("M,N,K", [(128, 128, 128), (256, 64, 32), (300, 200, 100), (513, 96, 1040), (1000, 40, 48), (130, 130, 2048),
                                   (384, 320, 16), (640, 1300, 144), (2048, 1536, 512), (77, 520, 272)])
def test_mn_major_operands_on_the_tensor_path(a_layout, b_layout, M, N, K):
    """Row-major B (the layout of the paper's printed GEMM listing, B[K][N]) and column-major A are consumed by the tensor
    kernels through MN-major descriptors: every tile width, ragged edges, one CTA per tile and CTA pairs."""
    import paper_2505_18574_b200 as i8
    pa = (-(M if a_layout == "col" else K)) % 16
    pb = (-(N if b_layout == "row" else K)) % 16
    p = inputs.make_gemm(M, N, K, 8000 + M + N + K, a_layout=a_layout, b_layout=b_layout, per_channel=1, relu=M % 2,
                         shift_lo=12, shift_hi=22, lda_pad=pa, ldb_pad=pb)
    want = H.gemm_oracle(p)
    for mode in (0, 2):
        i8.set_path(mode)
        got = H.gemm_gpu(p)
        assert i8.last_path() == (i8.PATH_TENSOR_2SM if mode == 2 else i8.PATH_TENSOR), (mode, i8.last_path())
        H.assert_same(got, want, f"{p.name} {a_layout}/{b_layout} mode {mode}")
    i8.set_path(0)
    assert i8.last_device_status() == 0


def test_mn_major_closed_form():
    """Oracle-independent: a one-hot A picks rows of a row-major B; with A stored column-major as well."""
    import paper_2505_18574_b200 as i8
    for a_layout in ("row", "col"):
        p = inputs.make_gemm(128, 384, 128, 4, a_layout=a_layout, b_layout="row", per_channel=0, relu=0, with_bias=False)
        p.A[:] = 0
        for i in range(128):
            k = (5 * i + 3) % 128
            if a_layout == "row":
                p.A[i, k] = 1
            else:
                p.A[k, i] = 1
        p.mult[:] = 1; p.shift[:] = 0
        got = H.gemm_gpu(p)
        assert i8.last_path() in TENSOR_PATHS
        want = np.stack([p.B[(5 * i + 3) % 128, :384] for i in range(128)])
        assert np.array_equal(got, want), a_layout


def test_unaligned_k_falls_back():
    p = inputs.make_gemm(65, 33, 37, 6, per_channel=0, relu=1, shared_shift=12)
    _both_paths(p, expect_tensor=False)


@pytest.mark.parametrize("mult,shift,relu", [(1, 0, 0), (-1, 0, 0), (2147483647, 31, 0), (-2147483648, 0, 0), (-2147483648, 31, 1),
                                              (0, 5, 0), (3, 1, 1), (65536, 16, 0), (-20000, 20, 1), (1, 31, 0)])
def test_extreme_scales(mult, shift, relu):
    p = inputs.make_gemm(128, 96, 64, 9, per_channel=0, relu=relu)
    p.mult[:] = mult; p.shift[:] = shift
    _both_paths(p)


def test_closed_forms_on_gpu():
    """Oracle-independent: all-ones operands give K everywhere; extreme constants give 2^27 at K = 8192."""
    import paper_2505_18574_b200 as i8
    for (a, b, K, mult, shift, expect) in [(1, 1, 96, 1, 0, 96), (-128, -128, 8192, 1, 21, 64), (-128, 127, 8192, 1, 20, -127)]:
        p = inputs.make_gemm(256, 128, K, 3, per_channel=0, relu=0, with_bias=False)
        p.A[:] = a; p.B[:] = b; p.mult[:] = mult; p.shift[:] = shift
        got = H.gemm_gpu(p)
        assert i8.last_path() in TENSOR_PATHS
        assert (got == expect).all(), (a, b, K, np.unique(got))


def test_config1a_full():
    p = inputs.config1(0)
    import paper_2505_18574_b200 as i8
    got = H.gemm_gpu(p)
    assert i8.last_path() == i8.PATH_TENSOR_2SM
    want = H.gemm_oracle(p)
    H.assert_same(got, want, p.name)
    H.not_degenerate(want)


@pytest.mark.parametrize("j", [1, 2])
def test_config1_large_full(j):
    """Full-size launch in the configuration the benchmark times, every element compared with the oracle (a few seconds
    of plain loops per problem on the host cores)."""
    import paper_2505_18574_b200 as i8
    p = inputs.config1(j)
    got = H.gemm_gpu(p)
    assert i8.last_path() == i8.PATH_TENSOR_2SM
    want = H.gemm_oracle(p)
    H.assert_same(got, want, p.name)
    H.not_degenerate(want)


def test_config4a_tall_skinny():
    import paper_2505_18574_b200 as i8
    p = inputs.config4a()
    got = H.gemm_gpu(p)
    assert i8.last_path() in (i8.PATH_TENSOR, i8.PATH_SMALL)
    want = H.gemm_oracle(p)
    H.assert_same(got, want, p.name)
    H.not_degenerate(want)


def test_bounded_wait_reports_timeout_and_context_survives():
    """A wait that nothing satisfies must end by itself with a status the host can read; the next call still works."""
    import time
    import paper_2505_18574_b200 as i8
    L = i8.lib()
    assert i8.last_device_status() == 0
    t0 = time.time()
    assert L.i8ops_selftest_bounded_wait(20, None) == 0
    assert i8.last_device_status() == 8            # I8_ERR_TIMEOUT
    assert time.time() - t0 < 5.0
    assert i8.last_device_status() == 0            # the record is cleared by the query
    p = inputs.make_gemm(128, 64, 64, 3, per_channel=0, relu=1)
    H.assert_same(H.gemm_gpu(p), H.gemm_oracle(p), "gemm after a timed-out wait")


@pytest.mark.parametrize("M,N,K,ldd_pad", [(128, 256, 128, 0), (300, 200, 112, 4), (513, 96, 1040, 0), (64, 40, 48, 3), (1000, 1024, 512, 0)])
def test_raw_accumulator_readout_and_split_k(M, N, K, ldd_pad):
    """gemm_i8_raw returns the int32 sums themselves; two accumulate calls over halves of K equal one call over all of K."""
    import torch
    import oracle
    import paper_2505_18574_b200 as i8
    p = inputs.make_gemm(M, N, K, 70 + M, per_channel=0, relu=0)
    want = oracle.gemm_acc(p.A, p.a_rs, 1, p.B, 1, p.b_cs, M, N, K).astype(np.int32)
    A = torch.from_numpy(p.A).cuda(); B = torch.from_numpy(p.B).cuda()
    for mode in (0, 1):
        i8.set_path(mode)
        Dbuf = torch.full((M, N + ldd_pad), 77, dtype=torch.int32, device="cuda")
        D = Dbuf[:, :N]
        i8.gemm_i8_raw(A, B.t(), D)
        assert i8.last_device_status() == 0
        assert i8.last_path() in (TENSOR_PATHS if mode == 0 else (i8.PATH_GENERIC,))
        H.assert_same(D.cpu().numpy(), want, f"raw mode {mode}")
        if ldd_pad:
            assert (Dbuf[:, N:] == 77).all()
        kh = (K // 32) * 16                     # split K at a multiple of 16 so both halves stay on the tensor path
        if kh:
            D.zero_()
            i8.gemm_i8_raw(A[:, :kh], B[:, :kh].t(), D, accumulate=True)
            i8.gemm_i8_raw(A[:, kh:], B[:, kh:].t(), D, accumulate=True)
            H.assert_same(D.cpu().numpy(), want, f"split-K accumulate mode {mode}")
    i8.set_path(0)


@pytest.mark.parametrize("M,N,K,lda_pad,ldb_pad,b_row_major", [(300, 200, 100, 3, 7, 0), (512, 384, 250, 0, 0, 1), (777, 130, 64, 5, 2, 1)])
def test_raw_and_float_scale_readouts_on_packed_operands(M, N, K, lda_pad, ldb_pad, b_row_major):
    """The other two read-outs with operands the tensor path cannot fetch in place (odd leading dimensions, K that is not a
    multiple of 16; for the float scale also row-major B): packed copies, tensor kernels, same results as the oracle."""
    import torch
    import oracle
    import paper_2505_18574_b200 as i8
    p = inputs.make_gemm(M, N, K, 4900 + M + K, per_channel=1, relu=1, lda_pad=lda_pad, ldb_pad=ldb_pad)
    acc = oracle.gemm_acc(p.A, p.a_rs, 1, p.B, 1, p.b_cs, M, N, K).astype(np.int32)
    rng = np.random.default_rng(M)
    scale = (rng.uniform(0.5, 1.0, size=N) * 2.0 ** rng.integers(-13, -9, size=N)).astype(np.float32)
    want_f = oracle.gemm_i8_fscale(p.A, p.a_rs, 1, p.B, 1, p.b_cs, N, p.bias, scale, 1, M, N, K, 1)
    A = torch.from_numpy(p.A).cuda()[:, :K]
    Bk = torch.from_numpy(p.B).cuda()[:, :K]                                  # (N, K) storage, K contiguous
    Bn = torch.from_numpy(np.ascontiguousarray(p.B[:, :K].T)).cuda()          # (K, N) storage, N contiguous
    bias, sc = torch.from_numpy(p.bias).cuda(), torch.from_numpy(scale).cuda()
    for mode in (0, 1):
        i8.set_path(mode)
        D = torch.full((M, N), 77, dtype=torch.int32, device="cuda")
        i8.gemm_i8_raw(A, Bk.t(), D)
        if (lda_pad or ldb_pad or K % 16) and mode == 0:
            assert i8.last_gemm_packed() and i8.last_path() in TENSOR_PATHS, (i8.last_gemm_packed(), i8.last_path())
        H.assert_same(D.cpu().numpy(), acc, f"raw, packed, mode {mode}")
        C = torch.full((M, N), 0x5A, dtype=torch.int8, device="cuda")
        i8.gemm_i8_fscale(A, Bn if b_row_major else Bk.t(), C, bias, sc, 1, 1)
        if mode == 0:
            assert i8.last_gemm_packed() == bool(b_row_major or lda_pad or ldb_pad or K % 16)
            assert i8.last_path() in TENSOR_PATHS, i8.last_path()
        else:
            assert i8.last_path() == i8.PATH_GENERIC
        H.assert_same(C.cpu().numpy(), want_f, f"float scale, packed, mode {mode}")
        assert i8.last_device_status() == 0
    i8.set_path(0)
    H.not_degenerate(want_f)


@pytest.mark.parametrize("M,N,K", [(512, 512, 128), (513, 600, 1040), (1000, 520, 272), (640, 1300, 144), (769, 1025, 48), (2048, 1536, 4096),
                                   (100, 300, 64), (256, 64, 96)])
def test_two_sm_kernel_shapes(M, N, K):
    """Shapes with M, N >= 512 run on the two-SM (cta_group::2) kernel: ragged edges in M, N and K, both epilogue forms."""
    pad = (-K) % 16
    for per_channel, relu, shift_hi in ((1, 0, 22), (0, 1, 18)):
        p = inputs.make_gemm(M, N, K, 2000 + M + N + K, per_channel=per_channel, relu=relu, shift_lo=12, shift_hi=shift_hi,
                             lda_pad=pad, ldb_pad=pad, ldc_pad=16 * per_channel)
        _both_paths(p, two_sm=True)
    p = inputs.make_gemm(M, N, K, 7, per_channel=0, relu=0, lda_pad=pad, ldb_pad=pad)
    p.mult[:] = -3; p.shift[:] = 0          # a scale outside the shift-32 form: the window form on the two-SM kernel
    _both_paths(p, two_sm=True)


@pytest.mark.parametrize("M,N,K", [
    (5000, 640, 256),      # 40 x 5 tiles of 128 x 128 over 148 CTAs: 29 or 30 workers per column, two rounds
    (3136, 2048, 512),     # the 1x1 convolution of the ResNet-like mix as a GEMM: 25 x 16 tiles, 9 or 10 workers per column
    (9001, 300, 64),       # ragged rows and columns, one K block
    (4100, 1000, 1104),    # nine K blocks, last one partial
    (20000, 520, 192),     # many rounds per worker
])
def test_column_sticky_tile_order(M, N, K):
    """Short-K problems with several tiles per CTA: each CTA keeps one block column (the epilogue constants are built
    once); every output tile must still be produced exactly once."""
    p = inputs.make_gemm(M, N, K, 77 + M + N, per_channel=1, relu=0)
    want = _both_paths(p)
    H.not_degenerate(want)


@pytest.mark.parametrize("M,N,K,ldc_pad", [(1, 13, 16, 3), (130, 200, 64, 8), (257, 328, 128, 0), (300, 135, 48, 9), (64, 1000, 32, 24),
                                           (513, 272, 256, 16), (100, 16, 16, 0)])
def test_wide_tiles_never_write_outside_c(M, N, K, ldc_pad):
    """The two-SM kernel (256-wide tiles, read-out through TMA stores where N is a multiple of 16) with ragged N, ragged M and a
    padded leading dimension: the harness checks the padding columns and the guard bytes around C."""
    import paper_2505_18574_b200 as i8
    p = inputs.make_gemm(M, N, K, 5 + M + N, per_channel=1, relu=0, ldc_pad=ldc_pad, shift_lo=10, shift_hi=16)
    want = H.gemm_oracle(p)
    for mode in (2, 0):
        i8.set_path(mode)
        H.assert_same(H.gemm_gpu(p), want, f"{p.name} mode {mode}")
    i8.set_path(0)


@pytest.mark.parametrize("seed", range(24))
def test_seeded_random_shapes_all_tile_orders(seed):
    """Medium-sized random shapes (several tiles per CTA, ragged edges, padded C) on the automatic path and on the forced
    two-SM path: exercises the raster and column-sticky tile orders, the TMA-store and direct read-outs and their edges."""
    import paper_2505_18574_b200 as i8
    rng = np.random.default_rng(1000 + seed)
    M = int(rng.integers(1, 6000)); N = int(rng.choice([16, 48, 64, 100, 128, 200, 256, 384, 520, 777, 1024, 1500]))
    K = 16 * int(rng.integers(1, 40))
    p = inputs.make_gemm(M, N, K, 2000 + seed, per_channel=int(rng.integers(0, 2)), relu=int(rng.integers(0, 2)),
                         ldc_pad=int(rng.choice([0, 0, 16, 5])), shift_lo=10, shift_hi=18)
    want = H.gemm_oracle(p)
    for mode in (0, 2):
        i8.set_path(mode)
        H.assert_same(H.gemm_gpu(p), want, f"{p.name} seed {seed} mode {mode}")
    i8.set_path(0)
    assert i8.last_device_status() == 0


@pytest.mark.parametrize("M,N,K,pinned", [(300, 200, 112, False), (2048, 512, 256, True), (5000, 384, 160, True), (8192, 256, 128, False)])
def test_host_buffer_variant(M, N, K, pinned):
    """gemm_i8_host: host buffers in, host buffer out (row chunks pipelined over three streams for M >= 2048)."""
    import torch
    import paper_2505_18574_b200 as i8
    p = inputs.make_gemm(M, N, K, 31 + M, per_channel=1, relu=1, shift_lo=12, shift_hi=20)
    want = H.gemm_oracle(p)
    mk = (lambda a: torch.from_numpy(a).pin_memory()) if pinned else (lambda a: torch.from_numpy(a))
    A, B, bias, mult, shift = mk(p.A), mk(p.B), mk(p.bias), mk(p.mult), mk(p.shift)
    C = torch.full((M, N), 0x5A, dtype=torch.int8)
    if pinned:
        C = C.pin_memory()
    for _ in range(2):                               # twice: the second call reuses the workspace, streams and events
        C.fill_(0x5A)
        i8.gemm_i8_host(A, B, C, bias, mult, shift, 1, 1)
        H.assert_same(C.numpy(), want, p.name + " host variant")
    assert i8.last_device_status() == 0


def test_recorded_class_plan_runs_and_is_reported():
    """Schedule reuse: a plan recorded on one square shape is what the library launches for the other square shapes near
    it (the plan query and the launch share one planning function), and the results stay bit-exact."""
    import paper_2505_18574_b200 as i8
    keys = ("tile_m", "tile_n", "stages", "cta_group", "raster_group", "sticky", "m_tiles", "n_tiles", "workers", "b_resident")
    try:
        i8.set_class_plan(0, base=(1024, 1024, 1024), tile_n=128, cta_group=1, raster_group=4, sticky=0)
        for (M, N, K) in [(1024, 1024, 1024), (512, 512, 512), (777, 600, 400)]:
            p = inputs.make_gemm(M, N, K + (-K) % 16, 4000 + M, per_channel=1, relu=0, shift_lo=12, shift_hi=20)
            got = H.gemm_gpu(p)
            assert i8.last_path() == i8.PATH_TENSOR
            ran, asked = i8.last_plan(), i8.plan_gemm(p.M, p.N, p.K)
            assert {k: ran[k] for k in keys} == {k: asked[k] for k in keys}
            assert (ran["tile_n"], ran["cta_group"], ran["raster_group"], ran["sticky"]) == (128, 1, 4, 0)
            H.assert_same(got, H.gemm_oracle(p), p.name)
        # CTA pairs recorded for a shape the crossover rule would leave on single CTAs
        i8.set_class_plan(0, base=(1024, 1024, 1024), tile_n=256, cta_group=2, raster_group=2)
        p = inputs.make_gemm(1000, 1100, 512, 4100, per_channel=1, relu=1, shift_lo=12, shift_hi=20)
        got = H.gemm_gpu(p)
        assert i8.last_path() == i8.PATH_TENSOR_2SM
        ran = i8.last_plan()
        assert (ran["tile_m"], ran["tile_n"], ran["cta_group"], ran["raster_group"], ran["stages"]) == (256, 256, 2, 2, 6)
        H.assert_same(got, H.gemm_oracle(p), p.name)
    finally:
        i8.set_class_plan(0, base=(8192, 8192, 8192), tile_n=256, cta_group=2, raster_group=16)
    # a shape the occupancy rule sends to the channel-major kernel: 12544 x 256 x 1152 (98 large tiles on 148 SMs)
    p = inputs.make_gemm(12544, 256, 1152, 4150, per_channel=1, relu=1)
    got = H.gemm_gpu(p)
    ran, asked = i8.last_plan(), i8.plan_gemm(p.M, p.N, p.K)
    assert i8.last_path() == i8.PATH_CHANNEL_MAJOR and ran["kernel"] == 1 and ran == asked
    assert ran["tile_n"] == 128 and ran["cta_group"] == 1 and ran["tile_m"] % 16 == 0
    assert ran["m_tiles"] * ran["tile_m"] >= p.M and ran["n_tiles"] == 2 and ran["workers"] <= 148
    H.assert_same(got, H.gemm_oracle(p), p.name)
    # without a recorded entry nearby, what ran is still what the query reports (config 1a: CTA pairs by the rule)
    p = inputs.make_gemm(2048, 2304, 1024, 4200, per_channel=1, relu=0)
    got = H.gemm_gpu(p)
    ran, asked = i8.last_plan(), i8.plan_gemm(p.M, p.N, p.K)
    assert {k: ran[k] for k in keys} == {k: asked[k] for k in keys}
    H.assert_same(got, H.gemm_oracle(p), p.name)


def test_tensor_map_cache_keys_on_the_address():
    """Encoded tensor maps are reused across calls; the same operands at another address must get their own maps."""
    import torch
    import paper_2505_18574_b200 as i8
    p = inputs.make_gemm(640, 384, 256, 4300, per_channel=1, relu=1, shift_lo=12, shift_hi=20)
    want = H.gemm_oracle(p)
    A1 = torch.from_numpy(p.A).cuda(); B1 = torch.from_numpy(p.B).cuda()
    A2 = A1.clone(); B2 = B1.clone()                       # same contents and geometry, other addresses
    assert A1.data_ptr() != A2.data_ptr() and B1.data_ptr() != B2.data_ptr()
    bias, mult, shift = (torch.from_numpy(a).cuda() for a in (p.bias, p.mult, p.shift))
    C = torch.empty((p.M, p.N), dtype=torch.int8, device="cuda")

    def run(A, B):
        C.fill_(0x5A)
        i8.gemm_i8(A, B.t(), C, bias, mult, shift, 1, 1)
        return C.cpu().numpy()

    H.assert_same(run(A1, B1), want, "first address")
    h0, m0 = i8.tmap_cache_stats()
    H.assert_same(run(A1, B1), want, "first address again")
    h1, m1 = i8.tmap_cache_stats()
    assert m1 == m0 and h1 >= h0 + 2, "the repeated call must reuse its maps (A and B; C too where the read-out uses TMA stores)"
    A2.zero_()                                             # were the first address's map reused, the result would not change
    got = run(A2, B1)
    h2, m2 = i8.tmap_cache_stats()
    assert m2 == m1 + 1 and h2 >= h1 + 1, "only A moved: one new map"
    assert not np.array_equal(got, want)
    A2.copy_(A1)
    H.assert_same(run(A2, B2), want, "second address")
    assert i8.last_device_status() == 0
