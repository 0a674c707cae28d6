"""Seeded synthetic inputs for the int8 GEMM / conv2d / batched-GEMM workloads.

This module only draws random tensors and names shapes.  It holds none of the
method's arithmetic (no products, no requantisation), so both the CPU oracle's
tests and the CUDA path's tests may use it without sharing any computation.

The shapes stand in for the paper's ResNet-50-derived Gemmini GEMM and
convolution benchmarks (Evaluation, "Gemmini Evaluation": GEMM, Convolution)
and for its fine-grained linear-algebra workload; the paper's own benchmark
files are not available, so every tensor is i.i.d. uniform:

* int8 operands and weights on [-128, 127]; convolution activations on
  [0, 127] (post-ReLU-like);
* int32 bias on [-2^15, 2^15);
* multiplier on [2^14, 2^15), one shared draw or one per output channel;
* shift 24 (shared) or an integer on [20, 28] per output channel.

Draw order per problem is fixed: A (or x), B (or w), bias, mult, shift, from one
``numpy.random.Generator(PCG64(seed))``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np


@dataclass
class GemmProblem:
    """C[M,N] = epilogue(A[M,K] . B[K,N]); strides are in elements."""
    name: str
    M: int
    N: int
    K: int
    A: np.ndarray            # int8, storage (M,K) if a_cs == 1 else (K,M)
    B: np.ndarray            # int8, storage (N,K) if b_rs == 1 else (K,N)
    a_rs: int
    a_cs: int
    b_rs: int
    b_cs: int
    ldc: int
    bias: Optional[np.ndarray]   # int32 [N] or None
    mult: np.ndarray             # int32 [1] or [N]
    shift: np.ndarray            # int32 [1] or [N]
    per_channel: int
    relu: int
    seed: int = 0


@dataclass
class ConvProblem:
    """y[N,P,Q,K] = epilogue(conv(x[N,H,W,C], w[K,R,S,C])), NHWC / KRSC."""
    name: str
    N: int
    H: int
    W: int
    C: int
    K: int
    R: int
    S: int
    stride_h: int
    stride_w: int
    pad_h: int
    pad_w: int
    x: np.ndarray
    w: np.ndarray
    bias: Optional[np.ndarray]
    mult: np.ndarray
    shift: np.ndarray
    per_channel: int
    relu: int
    seed: int = 0

    @property
    def P(self) -> int:
        return (self.H + 2 * self.pad_h - self.R) // self.stride_h + 1

    @property
    def Q(self) -> int:
        return (self.W + 2 * self.pad_w - self.S) // self.stride_w + 1


@dataclass
class BatchedProblem:
    """batch independent C_b[M,N] = epilogue(A_b[M,K] . B_b[K,N]), tight row-major."""
    name: str
    batch: int
    M: int
    N: int
    K: int
    A: np.ndarray            # int8 [batch, M, K]
    B: np.ndarray            # int8 [batch, K, N]
    bias: Optional[np.ndarray]   # int32 [batch, N] (per problem) or [N] (shared) or None
    bias_bs: int
    mult: np.ndarray
    shift: np.ndarray
    per_channel: int
    relu: int
    seed: int = 0


def _i8(rng, shape, lo=-128, hi=128):
    return rng.integers(lo, hi, size=shape, dtype=np.int8 if lo < 0 else np.int16).astype(np.int8)


def _requant_vectors(rng, n, per_channel, shift_lo=20, shift_hi=28, shared_shift=24):
    if per_channel:
        mult = rng.integers(1 << 14, 1 << 15, size=n, dtype=np.int32)
        shift = rng.integers(shift_lo, shift_hi + 1, size=n, dtype=np.int32)
    else:
        mult = rng.integers(1 << 14, 1 << 15, size=1, dtype=np.int32)
        shift = np.full(1, shared_shift, dtype=np.int32)
    return mult, shift


def make_gemm(M, N, K, seed, *, b_layout="col", a_layout="row", per_channel=0, relu=1,
              with_bias=True, name=None, shift_lo=20, shift_hi=28, shared_shift=24,
              lda_pad=0, ldb_pad=0, ldc_pad=0) -> GemmProblem:
    """Draw one GEMM problem.  ``b_layout='col'`` stores B as (N, K) with K contiguous."""
    rng = np.random.Generator(np.random.PCG64(seed))
    if a_layout == "row":
        A = _i8(rng, (M, K + lda_pad)); a_rs, a_cs = K + lda_pad, 1
    else:
        A = _i8(rng, (K, M + lda_pad)); a_rs, a_cs = 1, M + lda_pad
    if b_layout == "col":
        B = _i8(rng, (N, K + ldb_pad)); b_rs, b_cs = 1, K + ldb_pad
    else:
        B = _i8(rng, (K, N + ldb_pad)); b_rs, b_cs = N + ldb_pad, 1
    bias = rng.integers(-(1 << 15), 1 << 15, size=N, dtype=np.int32) if with_bias else None
    if not with_bias:
        rng.integers(0, 1, size=1)  # keep the stream position independent of with_bias
    mult, shift = _requant_vectors(rng, N, per_channel, shift_lo, shift_hi, shared_shift)
    return GemmProblem(name or f"gemm_{M}x{N}x{K}", M, N, K, A, B, a_rs, a_cs, b_rs, b_cs,
                       N + ldc_pad, bias, mult, shift, int(per_channel), int(relu), seed)


def make_conv(N, H, W, C, K, R, S, stride, pad, seed, *, per_channel=1, relu=1, with_bias=True,
              act_lo=0, act_hi=128, name=None) -> ConvProblem:
    rng = np.random.Generator(np.random.PCG64(seed))
    x = rng.integers(act_lo, act_hi, size=(N, H, W, C), dtype=np.int16).astype(np.int8)
    w = _i8(rng, (K, R, S, C))
    bias = rng.integers(-(1 << 15), 1 << 15, size=K, dtype=np.int32) if with_bias else None
    mult, shift = _requant_vectors(rng, K, per_channel)
    return ConvProblem(name or f"conv_{N}x{H}x{W}x{C}_k{K}_{R}x{S}_s{stride}", N, H, W, C, K, R, S,
                       stride, stride, pad, pad, x, w, bias, mult, shift, int(per_channel), int(relu), seed)


def make_batched(batch, M, N, K, seed, *, per_problem_bias=True, relu=1, name=None) -> BatchedProblem:
    rng = np.random.Generator(np.random.PCG64(seed))
    A = _i8(rng, (batch, M, K))
    B = _i8(rng, (batch, K, N))
    if per_problem_bias:
        bias = rng.integers(-(1 << 15), 1 << 15, size=(batch, N), dtype=np.int32); bias_bs = N
    else:
        bias = rng.integers(-(1 << 15), 1 << 15, size=N, dtype=np.int32); bias_bs = 0
    mult, shift = _requant_vectors(rng, N, 0)
    return BatchedProblem(name or f"batched_{batch}x{M}x{N}x{K}", batch, M, N, K, A, B, bias, bias_bs,
                          mult, shift, 0, int(relu), seed)


# ---------------------------------------------------------------------------------------------
# The five named workload configurations.  Seeds: config index, plus 100*j for sub-config j.
# ---------------------------------------------------------------------------------------------

GEMM_LARGE_SHAPES = [(4096, 4096, 4096), (8192, 8192, 8192), (16384, 4096, 8192)]
CONV_MIX = [  # (N, H, W, C, K, R, S, stride, pad)
    (64, 28, 28, 128, 256, 3, 3, 2, 1),
    (64, 14, 14, 256, 256, 3, 3, 1, 1),
    (64, 7, 7, 512, 2048, 1, 1, 1, 0),
]


def config0() -> GemmProblem:
    """256^3, A row-major, B col-major, shared mult, shift 24, ReLU on; seed 0."""
    return make_gemm(256, 256, 256, 0, per_channel=0, relu=1, name="cfg0_gemm_256")


def config1(j: int) -> GemmProblem:
    """Large GEMMs, per-output-channel mult/shift (shift on [20,28]), ReLU off."""
    M, N, K = GEMM_LARGE_SHAPES[j]
    return make_gemm(M, N, K, 1 + 100 * j, per_channel=1, relu=0, name=f"cfg1{'abc'[j]}_gemm_{M}x{N}x{K}")


def config2() -> ConvProblem:
    """Batch 32, 56x56x64 -> 64 filters 3x3, stride 1, pad 1, per-channel requant, ReLU on."""
    return make_conv(32, 56, 56, 64, 64, 3, 3, 1, 1, 2, name="cfg2_conv_56x56x64")


def config3(j: int) -> ConvProblem:
    """ResNet-like layer mix at batch 64, pad = R // 2."""
    N, H, W, C, K, R, S, st, pad = CONV_MIX[j]
    return make_conv(N, H, W, C, K, R, S, st, pad, 3 + 100 * j, name=f"cfg3{'abc'[j]}_conv_{H}x{W}x{C}_k{K}_{R}x{S}_s{st}")


def config4a() -> GemmProblem:
    """Tall-skinny M=262144, N=64, K=256; layouts and requant as config 0."""
    return make_gemm(262144, 64, 256, 4, per_channel=0, relu=1, name="cfg4a_skinny_262144x64x256")


def config4b() -> BatchedProblem:
    """16384 independent 64^3 GEMMs, tight row-major A/B/C, per-problem bias, shared mult/shift."""
    return make_batched(16384, 64, 64, 64, 104, name="cfg4b_batched_16384x64")


def extra_rowmajor_b() -> GemmProblem:
    """4096^3 with B stored row-major [K][N], the layout of the paper's printed Gemmini GEMM listing; otherwise as config 1a."""
    return make_gemm(4096, 4096, 4096, 501, b_layout="row", per_channel=1, relu=0, name="extra_gemm_4096cube_rowmajorB")


def extra_batched_128() -> BatchedProblem:
    """256 independent 128^3 products (above the paired 64^3 tile: one launch of the large-tile kernel per problem)."""
    return make_batched(256, 128, 128, 128, 502, name="extra_batched_256x128cube")


# ---------------------------------------------------------------------------------------------
# Shapes the paper itself prints (second workload): the Gemmini GEMM of its Code Examples
# appendix, the schedule-reuse table (square / column-dominant / row-dominant GEMMs, read as
# M x N x K with the listing's M=12544, K=256, N=64 for the column-dominant family), the
# ablation's convolution (batch 4, 3x3, 14x14, 256 -> 256 channels) and, as int8 stand-ins, the
# GEMM and conv2d shapes of its Trainium tables.  Seeds 200 + index; requantisation as config 1
# for the GEMMs and as config 2 for the convolutions.
# ---------------------------------------------------------------------------------------------
SWEEP_GEMMS = [  # (M, N, K)
    (12544, 64, 256), (1024, 1024, 1024), (512, 512, 512), (256, 256, 256), (6272, 64, 256), (12544, 64, 128),
    (128, 1024, 1024), (64, 1024, 1024), (32, 1024, 1024), (4096, 8192, 8192),
]
SWEEP_CONVS = [  # (N, H, W, C, K, R, S, stride, pad)
    (4, 14, 14, 256, 256, 3, 3, 1, 1),
    (16, 128, 128, 128, 512, 3, 3, 1, 1),
]


def sweep_gemm(i: int) -> GemmProblem:
    M, N, K = SWEEP_GEMMS[i]
    return make_gemm(M, N, K, 200 + i, per_channel=1, relu=0, name=f"sweep_gemm_{M}x{N}x{K}")


def sweep_conv(i: int) -> ConvProblem:
    N, H, W, C, K, R, S, st, pad = SWEEP_CONVS[i]
    return make_conv(N, H, W, C, K, R, S, st, pad, 300 + i, name=f"sweep_conv_{N}x{H}x{W}x{C}_k{K}_{R}x{S}")


# ---------------------------------------------------------------------------------------------
# Fine-grained linear algebra as the paper runs it: the TinyMPC primal-update forward pass
# (12 states, 4 inputs, NHORIZON = 5, fp32).  The paper's controller matrices are not available;
# the stand-ins are a stable random system: Adyn = I + 0.05*G (G standard normal), Bdyn = 0.1*G,
# Kinf = 0.3*G, initial states and d uniform on [-1, 1].  `batch` independent instances share
# the three matrices.
# ---------------------------------------------------------------------------------------------
@dataclass
class MpcProblem:
    name: str
    batch: int
    nhorizon: int
    Adyn: np.ndarray   # float32 [12, 12]
    Bdyn: np.ndarray   # float32 [12, 4]
    Kinf: np.ndarray   # float32 [4, 12]
    x0: np.ndarray     # float32 [batch, 12]
    d: np.ndarray      # float32 [batch, nhorizon, 4]
    seed: int = 0


def make_mpc(batch: int, nhorizon: int = 5, seed: int = 5, name=None) -> MpcProblem:
    rng = np.random.Generator(np.random.PCG64(seed))
    Adyn = (np.eye(12) + 0.05 * rng.standard_normal((12, 12))).astype(np.float32)
    Bdyn = (0.1 * rng.standard_normal((12, 4))).astype(np.float32)
    Kinf = (0.3 * rng.standard_normal((4, 12))).astype(np.float32)
    x0 = rng.uniform(-1.0, 1.0, size=(batch, 12)).astype(np.float32)
    d = rng.uniform(-1.0, 1.0, size=(batch, nhorizon, 4)).astype(np.float32)
    return MpcProblem(name or f"mpc_forward_{batch}x{nhorizon}", batch, nhorizon, Adyn, Bdyn, Kinf, x0, d, seed)
