"""Pins for the CPU oracle: facts fixed by the paper or by mathematics, none by the oracle itself.

Each ``pin_*`` function takes an ``oracle.Oracle`` and raises ``AssertionError`` when that oracle
violates the fact.  ``test_oracle_pins.py`` runs them on the real oracle (all must pass) and on
deliberately broken copies of ``oracle.c`` (each must be caught by at least one pin).
"""
from __future__ import annotations

import itertools
import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
I32_MIN, I32_MAX = -(1 << 31), (1 << 31) - 1


# ----------------------------------------------------------------------------- helpers (pure Python)
def py_requant(acc, bias, relu, mult, shift):
    """Python big-int model: Python's >> on ints is an exact floor shift at any magnitude."""
    t = acc + bias
    if relu:
        t = max(t, 0)
    r = (1 << (shift - 1)) if shift >= 1 else 0
    u = (t * mult + r) >> shift
    return max(-128, min(127, u))


def py_gemm_acc(A, B):
    """Brute-force triple loop over nested Python lists (exact integers)."""
    M, K, N = len(A), len(A[0]), len(B[0])
    return [[sum(A[m][k] * B[k][n] for k in range(K)) for n in range(N)] for m in range(M)]


def _c(a):
    return np.ascontiguousarray(a)


def _row_col(A, B):
    """A (M,K) row-major, B (K,N) given logically; store B column-major (N,K)."""
    return _c(A.astype(np.int8)), _c(B.T.astype(np.int8))


def _gemm(O, A, B, bias=None, mult=1, shift=0, relu=0, per_channel=0):
    """Logical A (M,K), B (K,N) -> C (M,N) through the oracle with row-major A, col-major B."""
    M, K = A.shape
    N = B.shape[1]
    As, Bs = _row_col(A, B)
    mult = np.atleast_1d(np.asarray(mult, dtype=np.int32))
    shift = np.atleast_1d(np.asarray(shift, dtype=np.int32))
    b = None if bias is None else _c(np.asarray(bias, dtype=np.int32))
    return O.gemm_i8(As, K, 1, Bs, 1, K, N, b, mult, shift, per_channel, M, N, K, relu)


def py_fl32(x):
    """Round an exact rational (fractions.Fraction) to the nearest IEEE-754 binary32 value, ties to even, with Python
    integers only (normal range; magnitudes here stay far from overflow and underflow).  Returns a Fraction."""
    from fractions import Fraction
    if x == 0:
        return Fraction(0)
    sign = -1 if x < 0 else 1
    a = abs(Fraction(x))
    e = a.numerator.bit_length() - a.denominator.bit_length()      # 2^e <= a < 2^(e+2): fix up below
    if Fraction(2) ** e > a:
        e -= 1
    if Fraction(2) ** (e + 1) <= a:
        e += 1
    ulp = Fraction(2) ** (e - 23)                                  # 24 significant bits
    q = a / ulp
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return sign * n * ulp


def py_rne_int(x):
    """Nearest integer of an exact rational, ties to even."""
    from fractions import Fraction
    n = x.numerator // x.denominator
    rem = x - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return n


def py_requant_fscale(acc, bias, relu, scale_num, scale_log2_den):
    """Exact-rational model of the float-scale read-out: fl32(fl32(t) * scale), nearest-even integer, clamp."""
    from fractions import Fraction
    t = acc + bias
    if relu:
        t = max(t, 0)
    scale = Fraction(scale_num, 1 << scale_log2_den)
    assert py_fl32(scale) == scale, "the scale must be a binary32 value"
    y = py_fl32(py_fl32(Fraction(t)) * scale)
    return max(-128, min(127, py_rne_int(y)))


# ----------------------------------------------------------------------------- float-scale pins
def pin_fscale_golden(O):
    """Hand-derived worked values (tests/golden/fscale_worked.txt)."""
    n = 0
    for line in open(os.path.join(GOLDEN, "fscale_worked.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        acc, bias, relu, num, lg, want = (int(v) for v in line.split())
        got, ovf = O.requant_fscale(acc, bias, relu, num / float(1 << lg))
        assert got == want and ovf == 0, (line, got)
        n += 1
    assert n >= 36


def pin_fscale_rational_model(O):
    """Against exact rational arithmetic with explicit binary32 roundings (Python integers), over edge accumulators,
    scales with full 24-bit mantissas and power-of-two scales; scale 1 is the saturating narrow; a power-of-two scale
    on a small accumulator is the round-to-even of an exact quotient."""
    accs = [0, 1, -1, 2, 3, -3, 127, 128, -128, -129, 255, 256, 1000, -1000, (1 << 23) + 1, (1 << 24) - 1, (1 << 24) + 1,
            -(1 << 24) - 3, (1 << 25) + 6, 3 * (1 << 25) + 3, 123456789, -987654321, I32_MAX, I32_MIN, I32_MAX - 64, 16777219]
    scales = [(1, 0), (1, 1), (3, 2), (1, 7), (5, 3), (16777215, 24), (16777215, 40), (8388609, 30), (11184811, 24), (1, 24),
              (12345677, 44), (3, 19), (13, 30), (-3, 2), (-16777215, 31), (1, 31)]
    rng = np.random.default_rng(11)
    accs = accs + [int(v) for v in rng.integers(-(1 << 31), 1 << 31, size=40)] + [int(v) for v in rng.integers(-4000, 4000, size=40)]
    for (num, lg) in scales:
        sc = num / float(1 << lg)
        for acc in accs:
            for relu in (0, 1):
                for bias in (0, -5):
                    if not (I32_MIN <= acc + bias <= I32_MAX):
                        continue
                    got, _ = O.requant_fscale(acc, bias, relu, sc)
                    assert got == py_requant_fscale(acc, bias, relu, num, lg), (acc, bias, relu, num, lg, got)
    for t in range(-300, 300):
        assert O.requant_fscale(t, 0, 0, 1.0)[0] == max(-128, min(127, t))
        q, r = divmod(t, 4)                         # t / 4 = q + r/4: nearest even
        want = q + (1 if r == 3 or (r == 2 and q % 2 == 1) else 0)
        assert O.requant_fscale(t, 0, 0, 0.25)[0] == max(-128, min(127, want)), t
    # monotone in t for a positive scale, antitone for a negative one; ReLU zeroes negatives; overflow flag
    for sc in (0.37, 1.5e-3, 2.0):
        prev = -128
        for t in range(-2000, 2000, 7):
            v = O.requant_fscale(t, 0, 0, sc)[0]
            assert v >= prev
            prev = v
            assert O.requant_fscale(t, 0, 1, sc)[0] == (v if t >= 0 else 0)
    assert O.requant_fscale(I32_MAX, 1, 0, 1.0)[1] == 1 and O.requant_fscale(I32_MAX, 0, 0, 1.0)[1] == 0


def pin_fscale_gemm(O):
    """The GEMM with the float-scale read-out: accumulators pinned by brute force elsewhere; here the read-out is applied
    per output column with the right scale and bias (per-channel and shared), and matches the element model."""
    rng = np.random.default_rng(12)
    M, N, K = 5, 7, 9
    A = rng.integers(-128, 128, size=(M, K)); B = rng.integers(-128, 128, size=(K, N))
    acc = py_gemm_acc(A.tolist(), B.tolist())
    bias = rng.integers(-3000, 3000, size=N).astype(np.int32)
    nums = [3, 5, 1, 7, 11, 13, 9]; lgs = [9, 10, 8, 11, 12, 12, 10]
    scale = np.array([n / float(1 << l) for n, l in zip(nums, lgs)], dtype=np.float32)
    As, Bs = _row_col(A, B)
    for relu in (0, 1):
        C = O.gemm_i8_fscale(As, K, 1, Bs, 1, K, N, bias, scale, 1, M, N, K, relu)
        for m in range(M):
            for n in range(N):
                assert C[m, n] == py_requant_fscale(acc[m][n], int(bias[n]), relu, nums[n], lgs[n]), (m, n)
        C1 = O.gemm_i8_fscale(As, K, 1, Bs, 1, K, N, None, scale[2:3].copy(), 0, M, N, K, relu)
        for m in range(M):
            for n in range(N):
                assert C1[m, n] == py_requant_fscale(acc[m][n], 0, relu, nums[2], lgs[2]), (m, n)
    # a transposed B (swapped strides) must change the result: storage order is honoured
    Bt = _c(B.astype(np.int8))                     # (K, N) row-major
    C2 = O.gemm_i8_fscale(As, K, 1, Bt, N, 1, N, bias, scale, 1, M, N, K, 0)
    C3 = O.gemm_i8_fscale(As, K, 1, Bs, 1, K, N, bias, scale, 1, M, N, K, 0)
    assert np.array_equal(C2, C3)


# ----------------------------------------------------------------------------- requant pins
def pin_requant_golden(O):
    """Hand-derived worked values (tests/golden/requant_worked.txt)."""
    n = 0
    for line in open(os.path.join(GOLDEN, "requant_worked.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        acc, bias, relu, mult, shift, exp = map(int, line.split())
        got, _ = O.requant(acc, bias, relu, mult, shift)
        assert got == exp, (line, got)
        n += 1
    assert n >= 40


def pin_requant_bigint_table(O):
    """Table against exact Python integers over edge accumulators, multipliers and all shifts."""
    accs = {0, 1, -1, I32_MIN, I32_MAX, I32_MIN + 1, I32_MAX - 1}
    for j in range(1, 31):
        for d in (-1, 0, 1):
            accs.add((1 << j) + d)
            accs.add(-(1 << j) + d)
    mults = [1, 2, 3, 1 << 14, (1 << 15) - 1, 20000, -1, -3, -(1 << 14), I32_MAX, I32_MIN, 0]
    for acc in sorted(accs):
        for mult in mults:
            for shift in range(0, 32):
                for relu in (0, 1):
                    got, ovf = O.requant(acc, 0, relu, mult, shift)
                    assert got == py_requant(acc, 0, relu, mult, shift), (acc, mult, shift, relu, got)
                    assert ovf == 0


def pin_requant_properties(O):
    rng = np.random.default_rng(11)
    # identity scale: mult = 2^s, shift = s  =>  clamp(acc)
    for s in range(0, 31):
        for acc in (-300, -129, -128, -1, 0, 1, 126, 127, 128, 4000):
            got, _ = O.requant(acc, 0, 0, 1 << s, s)
            assert got == max(-128, min(127, acc))
    # monotone non-decreasing in acc for mult >= 0; range; ReLU gives [0,127] for mult >= 0
    for _ in range(200):
        mult = int(rng.integers(0, 1 << 15))
        shift = int(rng.integers(0, 32))
        accs = np.sort(rng.integers(-(1 << 26), 1 << 26, size=64))
        prev = -129
        for a in accs:
            v, _ = O.requant(int(a), 0, 0, mult, shift)
            assert -128 <= v <= 127 and v >= prev
            prev = v
            vr, _ = O.requant(int(a), 0, 1, mult, shift)
            assert 0 <= vr <= 127
            # ReLU before or after the scale agree when mult >= 0 (monotone map through 0)
            assert vr == max(v, 0)
    # the bias enters as a plain addend of the accumulator
    for _ in range(200):
        acc = int(rng.integers(-(1 << 27), 1 << 27)); bias = int(rng.integers(-(1 << 15), 1 << 15))
        mult = int(rng.integers(1 << 14, 1 << 15)); shift = int(rng.integers(20, 29)); relu = int(rng.integers(0, 2))
        assert O.requant(acc, bias, relu, mult, shift)[0] == O.requant(acc + bias, 0, relu, mult, shift)[0]
    # overflow flag: exactly when acc + bias leaves int32
    assert O.requant(I32_MAX, 1, 0, 1, 0)[1] == 1
    assert O.requant(I32_MIN, -1, 0, 1, 0)[1] == 1
    assert O.requant(I32_MAX, 0, 0, 1, 0)[1] == 0
    assert O.requant(I32_MIN, 0, 0, 1, 0)[1] == 0


# ----------------------------------------------------------------------------- GEMM pins
def pin_gemm_bruteforce(O):
    """All shapes with M,N,K <= 4 plus a few odd ones, against Python-list integer loops."""
    rng = np.random.default_rng(5)
    shapes = list(itertools.product(range(1, 5), repeat=3)) + [(5, 3, 17), (17, 5, 3), (3, 17, 5), (7, 11, 13)]
    for (M, N, K) in shapes:
        A = rng.integers(-128, 128, size=(M, K)); B = rng.integers(-128, 128, size=(K, N))
        want = np.array(py_gemm_acc(A.tolist(), B.tolist()), dtype=np.int64)
        As, Bs = _row_col(A, B)
        got = O.gemm_acc(As, K, 1, Bs, 1, K, M, N, K)
        assert np.array_equal(got, want), (M, N, K)
        # the same logical product through every storage order of A and B
        At = _c(A.T.astype(np.int8)); Br = _c(B.astype(np.int8))
        assert np.array_equal(O.gemm_acc(At, 1, M, Br, N, 1, M, N, K), want)
        assert np.array_equal(O.gemm_acc(As, K, 1, Br, N, 1, M, N, K), want)
        assert np.array_equal(O.gemm_acc(At, 1, M, Bs, 1, K, M, N, K), want)


def pin_gemm_closed_forms(O):
    rng = np.random.default_rng(6)
    # identity: I . B = B  and  A . I = A
    n = 24
    B = rng.integers(-128, 128, size=(n, 19)); A = rng.integers(-128, 128, size=(13, n))
    I = np.eye(n, dtype=np.int64)
    As, Bs = _row_col(I, B)
    assert np.array_equal(O.gemm_acc(As, n, 1, Bs, 1, n, n, 19, n), B)
    As, Bs = _row_col(A, I)
    assert np.array_equal(O.gemm_acc(As, n, 1, Bs, 1, n, 13, n, n), A)
    # a shifted identity moves rows: (P B)[m] = B[m+1]
    Pm = np.eye(n, k=1, dtype=np.int64)
    As, Bs = _row_col(Pm, B)
    got = O.gemm_acc(As, n, 1, Bs, 1, n, n, 19, n)
    assert np.array_equal(got[:-1], B[1:]) and not got[-1].any()
    # constants: every entry K*a*b, including the extreme product of the int8 range
    for (a, b, K) in [(1, 1, 37), (-128, -128, 8192), (-128, 127, 8192), (3, -5, 100)]:
        A1 = np.full((3, K), a); B1 = np.full((K, 5), b)
        As, Bs = _row_col(A1, B1)
        got = O.gemm_acc(As, K, 1, Bs, 1, K, 3, 5, K)
        assert (got == K * a * b).all()
    assert 8192 * 128 * 128 == 1 << 27
    # numpy's integer matmul is a library routine for the same sum
    A = rng.integers(-128, 128, size=(33, 70)); B = rng.integers(-128, 128, size=(70, 29))
    As, Bs = _row_col(A, B)
    assert np.array_equal(O.gemm_acc(As, 70, 1, Bs, 1, 70, 33, 29, 70), A.astype(np.int64) @ B.astype(np.int64))


def pin_gemm_symmetries(O):
    rng = np.random.default_rng(7)
    M, N, K = 9, 14, 21
    A = rng.integers(-128, 128, size=(M, K)); B = rng.integers(-128, 128, size=(K, N))
    bias = rng.integers(-(1 << 15), 1 << 15, size=N)
    mult = rng.integers(1 << 14, 1 << 15, size=N); shift = rng.integers(12, 20, size=N)
    C = _gemm(O, A, B, bias, mult, shift, 0, 1)
    pk = rng.permutation(K); pm = rng.permutation(M); pn = rng.permutation(N)
    assert np.array_equal(_gemm(O, A[:, pk], B[pk, :], bias, mult, shift, 0, 1), C)            # sum order
    assert np.array_equal(_gemm(O, A[pm], B, bias, mult, shift, 0, 1), C[pm])                  # rows
    assert np.array_equal(_gemm(O, A, B[:, pn], bias[pn], mult[pn], shift[pn], 0, 1), C[:, pn])  # channels
    # per-channel vectors really are indexed by the output column, shared ones by nothing
    C0 = _gemm(O, A, B, bias, int(mult[3]), int(shift[3]), 0, 0)
    assert np.array_equal(C0[:, 3], C[:, 3])
    # padded leading dimensions do not change the result
    Ap = np.zeros((M, K + 5), dtype=np.int8); Ap[:, :K] = A
    Bp = np.zeros((N, K + 3), dtype=np.int8); Bp[:, :K] = B.T
    Cp = O.gemm_i8(Ap, K + 5, 1, Bp, 1, K + 3, N + 2, _c(bias.astype(np.int32)), _c(mult.astype(np.int32)),
                   _c(shift.astype(np.int32)), 1, M, N, K, 0)
    assert np.array_equal(Cp[:, :N], C) and not Cp[:, N:].any()


def pin_gemm_epilogue_on_matrix(O):
    """Whole-matrix epilogue against numpy int64 matmul + the big-int model, and the bias pin."""
    rng = np.random.default_rng(8)
    M, N, K = 12, 10, 64
    A = rng.integers(-128, 128, size=(M, K)); B = rng.integers(-128, 128, size=(K, N))
    bias = rng.integers(-(1 << 15), 1 << 15, size=N)
    acc = A.astype(np.int64) @ B.astype(np.int64)
    for relu in (0, 1):
        for (mult, shift) in [(1, 0), (20000, 10), (-7, 3), (32767, 24)]:
            C = _gemm(O, A, B, bias, mult, shift, relu, 0)
            want = [[py_requant(int(acc[m, n]), int(bias[n]), relu, mult, shift) for n in range(N)] for m in range(M)]
            assert np.array_equal(C, np.array(want))
    # the paper's printed GEMM case: no activation, scale 1.0, no bias  =>  saturate(A.B)
    C = _gemm(O, A, B, None, 1, 0, 0, 0)
    assert np.array_equal(C, np.clip(acc, -128, 127))
    # A = 0: the output is the scaled bias of its column, whatever B holds
    Z = np.zeros((M, K), dtype=np.int64)
    C = _gemm(O, Z, B, bias, 3, 9, 0, 0)
    want = np.array([py_requant(0, int(b), 0, 3, 9) for b in bias])
    assert (C == want[None, :]).all()
    # overflow report: K*2^14 stays in range at K = 8192, acc + bias beyond int32 is flagged
    As, Bs = _row_col(np.full((1, 8192), -128), np.full((8192, 1), -128))
    one = np.array([1], dtype=np.int32); zero = np.array([0], dtype=np.int32)
    _, ovf = O.gemm_i8(As, 8192, 1, Bs, 1, 8192, 1, np.array([I32_MAX - (1 << 27)], dtype=np.int32), one, zero,
                       0, 1, 1, 8192, 0, return_overflow=True)
    assert ovf == 0
    _, ovf = O.gemm_i8(As, 8192, 1, Bs, 1, 8192, 1, np.array([I32_MAX - (1 << 27) + 1], dtype=np.int32), one, zero,
                       0, 1, 1, 8192, 0, return_overflow=True)
    assert ovf == 1


# ----------------------------------------------------------------------------- batched pins
def pin_batched(O):
    rng = np.random.default_rng(9)
    batch, M, N, K = 5, 6, 7, 8
    A = rng.integers(-128, 128, size=(batch, M, K), dtype=np.int8)
    B = rng.integers(-128, 128, size=(batch, K, N), dtype=np.int8)
    bias = rng.integers(-(1 << 15), 1 << 15, size=(batch, N), dtype=np.int32)
    mult = np.array([21000], dtype=np.int32); shift = np.array([14], dtype=np.int32)
    C = O.batched_gemm_i8(A, K, 1, M * K, B, N, 1, K * N, N, M * N, bias, N, mult, shift, 0, batch, M, N, K, 1)
    C = C.reshape(batch, M, N)
    for b in range(batch):
        Cb = O.gemm_i8(_c(A[b]), K, 1, _c(B[b]), N, 1, N, _c(bias[b]), mult, shift, 0, M, N, K, 1)
        assert np.array_equal(C[b], Cb)
        acc = A[b].astype(np.int64) @ B[b].astype(np.int64)
        want = [[py_requant(int(acc[m, n]), int(bias[b, n]), 1, 21000, 14) for n in range(N)] for m in range(M)]
        assert np.array_equal(C[b], np.array(want))
    perm = rng.permutation(batch)
    Cp = O.batched_gemm_i8(_c(A[perm]), K, 1, M * K, _c(B[perm]), N, 1, K * N, N, M * N, _c(bias[perm]), N,
                           mult, shift, 0, batch, M, N, K, 1).reshape(batch, M, N)
    assert np.array_equal(Cp, C[perm])
    # a shared bias (stride 0) is the first bias row applied to every problem
    Cs = O.batched_gemm_i8(A, K, 1, M * K, B, N, 1, K * N, N, M * N, _c(bias[0]), 0, mult, shift, 0,
                           batch, M, N, K, 1).reshape(batch, M, N)
    for b in range(batch):
        Cb = O.gemm_i8(_c(A[b]), K, 1, _c(B[b]), N, 1, N, _c(bias[0]), mult, shift, 0, M, N, K, 1)
        assert np.array_equal(Cs[b], Cb)


# ----------------------------------------------------------------------------- convolution pins
def py_conv_acc(x, w, stride, pad):
    """Brute-force direct convolution on nested lists / small arrays with Python integers."""
    N, H, W, C = x.shape
    K, R, S, _ = w.shape
    P = (H + 2 * pad - R) // stride + 1
    Q = (W + 2 * pad - S) // stride + 1
    out = np.zeros((N, P, Q, K), dtype=np.int64)
    for n in range(N):
        for p in range(P):
            for q in range(Q):
                for k in range(K):
                    acc = 0
                    for r in range(R):
                        for s in range(S):
                            h = p * stride - pad + r
                            ww = q * stride - pad + s
                            if 0 <= h < H and 0 <= ww < W:
                                for c in range(C):
                                    acc += int(x[n, h, ww, c]) * int(w[k, r, s, c])
                    out[n, p, q, k] = acc
    return out


def _conv_raw(O, x, w, stride, pad, bias=None, mult=1, shift=0, relu=0, per_channel=0, **kw):
    N, H, W, C = x.shape
    K, R, S, _ = w.shape
    mult = np.atleast_1d(np.asarray(mult, dtype=np.int32)); shift = np.atleast_1d(np.asarray(shift, dtype=np.int32))
    b = None if bias is None else _c(np.asarray(bias, dtype=np.int32))
    return O.conv2d_i8(_c(x.astype(np.int8)), _c(w.astype(np.int8)), b, mult, shift, per_channel,
                       N, H, W, C, K, R, S, stride, stride, pad, pad, relu, **kw)


def pin_conv_bruteforce(O):
    """Small values keep the raw sum inside int8 so that scale 1 exposes the accumulator itself."""
    rng = np.random.default_rng(10)
    cases = [(1, 4, 4, 2, 3, 3, 3, 1, 1), (2, 5, 5, 3, 2, 3, 3, 2, 1), (2, 4, 5, 1, 2, 3, 3, 2, 1),
             (1, 5, 4, 2, 2, 1, 1, 1, 0), (1, 6, 6, 2, 2, 3, 3, 1, 0), (2, 5, 6, 2, 3, 1, 1, 2, 0),
             (1, 7, 7, 1, 1, 5, 5, 2, 2)]
    for (N, H, W, C, K, R, S, st, pad) in cases:
        x = rng.integers(-3, 4, size=(N, H, W, C)); w = rng.integers(-2, 3, size=(K, R, S, C))
        want = py_conv_acc(x, w, st, pad)
        assert np.abs(want).max() <= 127
        got = _conv_raw(O, x, w, st, pad)
        assert got.shape == want.shape and np.array_equal(got, want), (N, H, W, C, K, R, S, st, pad)
    # full-range values with a real scale, against the brute force + big-int epilogue
    x = rng.integers(0, 128, size=(2, 5, 5, 3)); w = rng.integers(-128, 128, size=(4, 3, 3, 3))
    bias = rng.integers(-(1 << 15), 1 << 15, size=4); mult = rng.integers(1 << 14, 1 << 15, size=4)
    shift = rng.integers(20, 25, size=4)
    for st in (1, 2):
        acc = py_conv_acc(x, w, st, 1)
        got = _conv_raw(O, x, w, st, 1, bias, mult, shift, 1, 1)
        want = np.zeros_like(acc)
        for idx in np.ndindex(acc.shape):
            k = idx[3]
            want[idx] = py_requant(int(acc[idx]), int(bias[k]), 1, int(mult[k]), int(shift[k]))
        assert np.array_equal(got, want)


def pin_conv_closed_forms(O):
    rng = np.random.default_rng(12)
    # 1x1, stride 1, pad 0 is a GEMM over pixels
    N, H, W, C, K = 2, 5, 6, 7, 4
    x = rng.integers(-128, 128, size=(N, H, W, C)); w = rng.integers(-128, 128, size=(K, 1, 1, C))
    bias = rng.integers(-(1 << 15), 1 << 15, size=K); mult = rng.integers(1 << 14, 1 << 15, size=K)
    shift = rng.integers(14, 20, size=K)
    y = _conv_raw(O, x, w, 1, 0, bias, mult, shift, 1, 1)
    Cg = _gemm(O, x.reshape(-1, C), w.reshape(K, C).T, bias, mult, shift, 1, 1)
    assert np.array_equal(y.reshape(-1, K), Cg)
    # delta filter: one 1 at tap (r,s), channel c -> filter k: the output is the input shifted by
    # (r - pad, s - pad), zero outside the image, sub-sampled by the stride (no kernel flip)
    N, H, W, C, K = 1, 6, 7, 3, 3
    x = rng.integers(-100, 101, size=(N, H, W, C))
    for st in (1, 2):
        for (r, s) in itertools.product(range(3), repeat=2):
            w = np.zeros((K, 3, 3, C), dtype=np.int64)
            for k in range(K):
                w[k, r, s, (k + 1) % C] = 1
            y = _conv_raw(O, x, w, st, 1)
            P = (H + 2 - 3) // st + 1; Q = (W + 2 - 3) // st + 1
            assert y.shape == (N, P, Q, K)
            for p in range(P):
                for q in range(Q):
                    h = p * st - 1 + r; ww = q * st - 1 + s
                    for k in range(K):
                        want = x[0, h, ww, (k + 1) % C] if (0 <= h < H and 0 <= ww < W) else 0
                        assert y[0, p, q, k] == want, (st, r, s, p, q, k)
    # all ones, 3x3 pad 1 stride 1: interior 9C, edges 6C, corners 4C
    N, H, W, C, K = 1, 5, 6, 2, 2
    y = _conv_raw(O, np.ones((N, H, W, C)), np.ones((K, 3, 3, C)), 1, 1)
    assert (y[0, 1:-1, 1:-1] == 9 * C).all()
    assert (y[0, 0, 1:-1] == 6 * C).all() and (y[0, -1, 1:-1] == 6 * C).all()
    assert (y[0, 1:-1, 0] == 6 * C).all() and (y[0, 1:-1, -1] == 6 * C).all()
    assert y[0, 0, 0, 0] == 4 * C and y[0, -1, -1, 1] == 4 * C and y[0, 0, -1, 0] == 4 * C
    # output extent: floor((H + 2 pad - R) / stride) + 1
    assert _conv_raw(O, np.ones((1, 28, 28, 1)), np.ones((1, 3, 3, 1)), 2, 1).shape == (1, 14, 14, 1)
    assert _conv_raw(O, np.ones((1, 7, 7, 1)), np.ones((1, 1, 1, 1)), 1, 0).shape == (1, 7, 7, 1)
    # image slabs: computing [n0, n1) writes exactly those images
    x = rng.integers(0, 128, size=(3, 4, 4, 2)); w = rng.integers(-128, 128, size=(2, 3, 3, 2))
    full = _conv_raw(O, x, w, 1, 1, None, 9000, 12)
    part = _conv_raw(O, x, w, 1, 1, None, 9000, 12, n_begin=1, n_end=2)
    assert np.array_equal(part[1], full[1]) and not part[0].any() and not part[2].any()


ALL_PINS = [pin_fscale_golden, pin_fscale_rational_model, pin_fscale_gemm, pin_requant_golden, pin_requant_bigint_table, pin_requant_properties, pin_gemm_bruteforce,
            pin_gemm_closed_forms, pin_gemm_symmetries, pin_gemm_epilogue_on_matrix, pin_batched,
            pin_conv_bruteforce, pin_conv_closed_forms]
