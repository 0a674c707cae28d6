"""CPU-side checks of the boundary: the library loads, exports every declared symbol, and rejects bad
arguments before anything is launched (no GPU needed: validation precedes every CUDA call)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2505_18574_b200 import build
    build.build()
    from paper_2505_18574_b200 import binding
    return binding.lib()


def test_exports_every_declared_symbol(L):
    from paper_2505_18574_b200 import binding
    header = open(os.path.join(ROOT, "include", "i8ops.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b([A-Za-z_][A-Za-z0-9_]*)\s*\(", header))
    declared = {d for d in declared if d.startswith(("gemm_", "conv2d_", "batched_", "i8_", "i8ops_"))}
    assert {"gemm_i8", "conv2d_i8", "batched_gemm_i8", "gemm_i8_host", "i8_status_string",
            "i8ops_last_device_status"} <= declared
    for name in declared:
        assert hasattr(L, name), f"{name} declared in i8ops.h but not exported"
        assert name in binding.SIGNATURES, f"{name} has no binding signature"


def test_status_strings(L):
    assert L.i8_status_string(0) == b"ok"
    for s in range(1, 9):
        assert L.i8_status_string(s) not in (b"ok", b"unknown status")
    assert L.i8_status_string(99) == b"unknown status"
    assert L.i8ops_version() >= 1


def test_gemm_argument_validation(L):
    P = ctypes.c_void_p
    buf = (ctypes.c_int8 * 4096)()
    v32 = (ctypes.c_int32 * 64)()
    a = ctypes.addressof(buf); q = ctypes.addressof(v32)

    def call(A=a, a_rs=16, a_cs=1, B=a, b_rs=1, b_cs=16, C=a, ldc=16, mult=q, shift=q, M=16, N=16, K=16):
        return L.gemm_i8(P(A) if A else None, a_rs, a_cs, P(B) if B else None, b_rs, b_cs, P(C) if C else None, ldc,
                         None, P(mult) if mult else None, P(shift) if shift else None, 0, M, N, K, 0, None)
    assert call(M=-1) == 2 and call(N=-1) == 2 and call(K=-1) == 2          # I8_ERR_SHAPE
    assert call(K=65537) == 5                                                # I8_ERR_RANGE
    assert call(A=None) == 1 and call(B=None) == 1 and call(C=None) == 1     # I8_ERR_NULL
    assert call(mult=None) == 1 and call(shift=None) == 1
    assert call(a_rs=2, a_cs=2) == 3 and call(b_rs=3, b_cs=16) == 3          # I8_ERR_STRIDE: no unit stride
    assert call(a_rs=8) == 3 and call(b_cs=8) == 3 and call(ldc=8) == 3      # leading dimension too small
    assert call(a_rs=-16) == 3
    assert call(M=0) == 0 and call(N=0) == 0                                 # empty problems are fine
    assert L.i8ops_last_path() == 0


def test_float_scale_and_probe_argument_validation(L):
    P = ctypes.c_void_p
    buf = (ctypes.c_int8 * 4096)()
    f32 = (ctypes.c_float * 64)()
    a = P(ctypes.addressof(buf)); q = P(ctypes.addressof(f32))

    def call(A=a, B=a, C=a, scale=q, M=16, N=16, K=16, a_rs=16, b_cs=16, ldc=16):
        return L.gemm_i8_fscale(A, a_rs, 1, B, 1, b_cs, C, ldc, None, scale, 0, M, N, K, 0, None)
    assert call(scale=None) == 1 and call(A=None) == 1 and call(C=None) == 1          # I8_ERR_NULL
    assert call(M=-1) == 2 and call(K=65537) == 5 and call(ldc=8) == 3 and call(a_rs=8) == 3
    assert call(M=0) == 0 and call(N=0) == 0
    # the issue-rate probe checks its ranges before any CUDA call
    assert L.i8ops_probe_mma_rate(256, 4096, 1, None, None) == 1
    for bad in ((8, 4096, 1), (272, 4096, 1), (250, 4096, 1), (256, 100, 1), (256, 32, 1), (256, 4096, 0)):
        assert L.i8ops_probe_mma_rate(bad[0], bad[1], bad[2], a, None) == 5, bad


def test_batched_and_conv_argument_validation(L):
    P = ctypes.c_void_p
    buf = (ctypes.c_int8 * 4096)()
    v32 = (ctypes.c_int32 * 64)()
    a = P(ctypes.addressof(buf)); q = P(ctypes.addressof(v32))
    assert L.batched_gemm_i8(a, 16, 1, 256, a, 16, 1, 256, a, 16, 256, None, 0, q, q, 0, -1, 16, 16, 16, 0, None) == 2
    assert L.batched_gemm_i8(a, 16, 1, -1, a, 16, 1, 256, a, 16, 256, None, 0, q, q, 0, 2, 16, 16, 16, 0, None) == 3
    assert L.batched_gemm_i8(a, 16, 1, 256, a, 16, 1, 256, a, 16, 256, None, 0, q, q, 0, 0, 16, 16, 16, 0, None) == 0

    def conv(x=a, w=a, y=a, N=1, H=8, W=8, C=4, K=4, R=3, S=3, sh=1, sw=1, ph=1, pw=1, mult=q):
        return L.conv2d_i8(x, w, y, None, mult, q, 0, N, H, W, C, K, R, S, sh, sw, ph, pw, 0, None)
    assert conv(N=0) == 2 and conv(C=0) == 2 and conv(R=0) == 2
    assert conv(sh=0) == 6 and conv(pw=-1) == 6
    assert conv(H=1, ph=0) == 2                     # filter taller than the padded image: empty output
    assert conv(C=8192, R=3, S=3) == 5              # R*S*C > 65536
    assert conv(x=None) == 1 and conv(mult=None) == 1


def test_host_variant_checks_shift(L):
    import numpy as np
    A = np.zeros((4, 16), np.int8); B = np.zeros((4, 16), np.int8); C = np.zeros((4, 4), np.int8)
    mult = np.ones(1, np.int32)
    for bad in (-1, 32):
        shift = np.array([bad], np.int32)
        assert L.gemm_i8_host(A.ctypes.data, B.ctypes.data, C.ctypes.data, None, mult.ctypes.data, shift.ctypes.data,
                              0, 4, 4, 16, 0, None) == 5


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    from paper_2505_18574_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError):
        binding.lib()


def test_tile_plan_and_class_reuse(L):
    """Host-side plan query and the schedule-reuse analogue: shapes of one aspect class share a recorded tile."""
    from paper_2505_18574_b200 import binding
    # the paper's reuse table: base shape and its two reuse targets per class (M x N x K)
    table = {0: [(1024, 1024, 1024), (512, 512, 512), (256, 256, 256)],
             1: [(12544, 64, 256), (6272, 64, 256), (12544, 64, 128)],
             2: [(128, 1024, 1024), (64, 1024, 1024), (32, 1024, 1024)]}
    for cls, shapes in table.items():
        for (M, N, K) in shapes:
            pl = binding.plan_gemm(M, N, K)
            assert pl["shape_class"] == cls and pl["tile_m"] == 128 and pl["tile_n"] in (64, 128, 256)
            assert pl["m_tiles"] == -(-M // 128) and pl["n_tiles"] == -(-N // pl["tile_n"])
            assert pl["waves"] == -(-(pl["m_tiles"] * pl["n_tiles"]) // 148)
    assert binding.plan_gemm(12544, 64, 256)["b_resident"] == 1 and binding.plan_gemm(8192, 8192, 8192)["b_resident"] == 0
    big = binding.plan_gemm(8192, 8192, 8192)
    # the large square GEMMs run on CTA pairs: 256 x 256 tiles, six ring slots, one worker per pair of SMs
    assert (big["tile_m"], big["tile_n"], big["cta_group"], big["stages"], big["workers"]) == (256, 256, 2, 6, 74)
    assert big["m_tiles"] == 32 and big["n_tiles"] == 32 and big["waves"] == -(-1024 // 74) and big["raster_group"] == 16
    small = binding.plan_gemm(256, 256, 256)
    assert small["cta_group"] == 1 and small["tile_m"] == 128 and small["workers"] == small["m_tiles"] * small["n_tiles"]
    skinny = binding.plan_gemm(262144, 64, 256)
    assert (skinny["tile_n"], skinny["cta_group"], skinny["stages"], skinny["b_resident"], skinny["workers"]) == (64, 1, 6, 1, 148)
    sticky = binding.plan_gemm(3136, 2048, 512)         # short K, several tiles per worker: column-sticky order
    assert sticky["sticky"] == 1 and sticky["tile_n"] == 128
    try:
        base = binding.plan_gemm(1024, 1024, 1024)["tile_n"]
        other = 128 if base != 128 else 64
        binding.set_class_tile(0, other)                       # record a schedule for the square class ...
        for (M, N, K) in table[0]:
            assert binding.plan_gemm(M, N, K)["tile_n"] == other   # ... and every square shape reuses it
        assert binding.plan_gemm(12544, 64, 256)["tile_n"] == 64   # other classes are untouched
        binding.set_class_tile(1, 256)                         # wider than a 64-column problem: ignored
        assert binding.plan_gemm(12544, 64, 256)["tile_n"] == 64
    finally:
        for c in range(3):
            binding.set_class_tile(c, 0)
    assert binding.plan_gemm(1024, 1024, 1024)["tile_n"] == base
    assert L.i8ops_set_class_tile(3, 64) == 5 and L.i8ops_set_class_tile(0, 100) == 5
    # a full class entry: (tile, cta_group, raster group, sticky) found on a base shape is reused by shapes within a
    # factor of four of it, and by no others
    try:
        binding.set_class_plan(0, base=(1024, 1024, 1024), tile_n=128, cta_group=1, raster_group=4, sticky=0)
        for (M, N, K) in table[0]:
            pl = binding.plan_gemm(M, N, K)
            assert (pl["tile_n"], pl["cta_group"], pl["raster_group"], pl["sticky"]) == (128, 1, 4, 0)
        far = binding.plan_gemm(8192, 8192, 8192)
        assert (far["tile_n"], far["cta_group"], far["raster_group"]) == (256, 2, 16)      # too far from the base: the rule decides
        binding.set_class_plan(0, base=(4096, 4096, 4096), cta_group=1, tile_n=256)
        assert binding.plan_gemm(4096, 4096, 4096)["cta_group"] == 1 and binding.plan_gemm(4096, 4096, 4096)["tile_m"] == 128
    finally:
        binding.set_class_plan(0, base=(8192, 8192, 8192), tile_n=256, cta_group=2, raster_group=16)    # the seeded entries
        binding.set_class_plan(1, base=(262144, 64, 256), tile_n=64, cta_group=1, raster_group=16)
    assert L.i8ops_set_class_plan(0, 1024, 0, 1024, 128, 0, 0, -1) == 5      # a base shape is all three extents or none
    assert L.i8ops_set_class_plan(0, 0, 0, 0, 128, 2, 0, -1) == 5            # CTA pairs imply 256-wide tiles
    assert L.i8ops_set_class_plan(0, 0, 0, 0, 0, 3, 0, -1) == 5 and L.i8ops_set_class_plan(0, 0, 0, 0, 0, 0, 65, -1) == 5
    assert L.i8ops_plan_gemm(0, 1, 1, 148, None) == 1
