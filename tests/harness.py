"""Glue for the parity tests: run one seeded problem through the CUDA library (via its C ABI binding)
and through the CPU oracle, and hand back both results as numpy arrays."""
from __future__ import annotations

import numpy as np


def _t(a, dev="cuda"):
    import torch
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dev)


# ------------------------------------------------------------------------------------------------ GEMM
def gemm_gpu(p, guard: int = 64):
    """Returns C (M, N) from the CUDA path; also checks guard bytes around C stayed untouched."""
    import torch
    import paper_2505_18574_b200 as i8
    A = _t(p.A); B = _t(p.B)
    Av = A if p.a_cs == 1 else A.t()            # logical (M, K)
    Bv = B.t() if p.b_rs == 1 else B            # logical (K, N)
    Av = Av[:, :p.K] if p.a_cs == 1 else Av[:p.M, :]
    Bv = Bv[:p.K, :] if p.b_rs == 1 else Bv[:, :p.N]
    Av = Av[:p.M, :p.K]; Bv = Bv[:p.K, :p.N]
    buf = torch.full((p.M * p.ldc + 2 * guard,), 0x5A, dtype=torch.int8, device="cuda")
    C = buf[guard:guard + p.M * p.ldc].view(p.M, p.ldc)[:, :p.N]
    i8.gemm_i8(Av, Bv, C, _t(p.bias), _t(p.mult), _t(p.shift), p.per_channel, p.relu)
    st = i8.last_device_status()
    assert st == 0, f"device status {st}"
    host = buf.cpu().numpy()
    assert (host[:guard] == 0x5A).all() and (host[guard + p.M * p.ldc:] == 0x5A).all(), "guard bytes overwritten"
    full = host[guard:guard + p.M * p.ldc].reshape(p.M, p.ldc)
    if p.ldc > p.N:
        assert (full[:, p.N:] == 0x5A).all(), "padding columns of C overwritten"
    return full[:, :p.N].copy()


def gemm_oracle(p):
    import oracle
    C = oracle.gemm_i8(p.A, p.a_rs, p.a_cs, p.B, p.b_rs, p.b_cs, p.ldc, p.bias, p.mult, p.shift, p.per_channel,
                       p.M, p.N, p.K, p.relu)
    return C[:, :p.N]


# ------------------------------------------------------------------------------------------------ batched
def batched_gpu(p):
    import torch
    import paper_2505_18574_b200 as i8
    A = _t(p.A); B = _t(p.B)
    C = torch.full((p.batch, p.M, p.N), 0x5A, dtype=torch.int8, device="cuda")
    i8.batched_gemm_i8(A, B, C, _t(p.bias), _t(p.mult), _t(p.shift), p.per_channel, p.relu)
    assert i8.last_device_status() == 0
    return C.cpu().numpy()


def batched_oracle(p):
    import oracle
    C = oracle.batched_gemm_i8(p.A, p.K, 1, p.M * p.K, p.B, p.N, 1, p.K * p.N, p.N, p.M * p.N, p.bias, p.bias_bs,
                               p.mult, p.shift, p.per_channel, p.batch, p.M, p.N, p.K, p.relu)
    return C.reshape(p.batch, p.M, p.N)


# ------------------------------------------------------------------------------------------------ conv
def conv_gpu(p, guard: int = 64):
    import torch
    import paper_2505_18574_b200 as i8
    n_out = p.N * p.P * p.Q * p.K
    buf = torch.full((n_out + 2 * guard,), 0x5A, dtype=torch.int8, device="cuda")
    y = buf[guard:guard + n_out].view(p.N, p.P, p.Q, p.K)
    i8.conv2d_i8(_t(p.x), _t(p.w), y, _t(p.bias), _t(p.mult), _t(p.shift), p.per_channel, p.relu,
                 (p.stride_h, p.stride_w), (p.pad_h, p.pad_w))
    assert i8.last_device_status() == 0
    host = buf.cpu().numpy()
    assert (host[:guard] == 0x5A).all() and (host[guard + n_out:] == 0x5A).all(), "guard bytes overwritten"
    return host[guard:guard + n_out].reshape(p.N, p.P, p.Q, p.K).copy()


def conv_oracle(p, n_begin=0, n_end=None):
    import oracle
    return oracle.conv2d_i8(p.x, p.w, p.bias, p.mult, p.shift, p.per_channel, p.N, p.H, p.W, p.C, p.K, p.R, p.S,
                            p.stride_h, p.stride_w, p.pad_h, p.pad_w, p.relu, n_begin, n_end)


def assert_same(got: np.ndarray, want: np.ndarray, what: str = ""):
    if got.shape != want.shape:
        raise AssertionError(f"{what}: shape {got.shape} vs {want.shape}")
    if not np.array_equal(got, want):
        bad = np.argwhere(got != want)
        first = tuple(bad[0])
        raise AssertionError(f"{what}: {len(bad)} of {got.size} elements differ; first at {first}: "
                             f"got {got[first]} want {want[first]}; rows {sorted(set(bad[:, 0].tolist()))[:8]} "
                             f"cols {sorted(set(bad[:, -1].tolist()))[:8]}")


def not_degenerate(C: np.ndarray):
    """Parity on an all-saturated or all-zero output would prove little."""
    sat = ((C == 127) | (C == -128) | (C == 0)).mean()
    assert sat < 0.98, f"output almost entirely saturated/zero ({sat:.3f})"
