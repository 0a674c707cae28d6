"""ctypes front end of ``oracle.c`` (plain C loops; see that file's header for what each
function computes and which passage of the paper defines it).

TEST INFRASTRUCTURE: arguments are numpy arrays in host memory; nothing here touches a GPU and
nothing here is imported by the CUDA path.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")

_i8p = ctypes.POINTER(ctypes.c_int8)
_i32p = ctypes.POINTER(ctypes.c_int32)
_i64p = ctypes.POINTER(ctypes.c_int64)
_i64 = ctypes.c_int64
_int = ctypes.c_int


def build(force: bool = False) -> str:
    """Compile ``oracle.c`` into ``liboracle.so`` beside it (gcc, OpenMP over output rows)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11",
               "-Wall", "-Wextra", "-o", _SO, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def _bind(path: str):
    L = ctypes.CDLL(path)
    L.oracle_requant.restype = ctypes.c_int32
    L.oracle_requant.argtypes = [_i64, ctypes.c_int32, _int, ctypes.c_int32, ctypes.c_int32,
                                 ctypes.POINTER(_int)]
    L.oracle_requant_fscale.restype = ctypes.c_int32
    L.oracle_requant_fscale.argtypes = [_i64, ctypes.c_int32, _int, ctypes.c_float, ctypes.POINTER(_int)]
    L.oracle_gemm_i8_fscale.restype = _int
    L.oracle_gemm_i8_fscale.argtypes = [_i8p, _i64, _i64, _i8p, _i64, _i64, _i8p, _i64, _i32p,
                                        ctypes.POINTER(ctypes.c_float), _int, _int, _int, _int, _int]
    L.oracle_gemm_acc.restype = None
    L.oracle_gemm_acc.argtypes = [_i8p, _i64, _i64, _i8p, _i64, _i64, _i64p, _int, _int, _int]
    L.oracle_gemm_i8.restype = _int
    L.oracle_gemm_i8.argtypes = [_i8p, _i64, _i64, _i8p, _i64, _i64, _i8p, _i64,
                                 _i32p, _i32p, _i32p, _int, _int, _int, _int, _int]
    L.oracle_batched_gemm_i8.restype = _int
    L.oracle_batched_gemm_i8.argtypes = [_i8p, _i64, _i64, _i64, _i8p, _i64, _i64, _i64,
                                         _i8p, _i64, _i64, _i32p, _i64, _i32p, _i32p, _int,
                                         _int, _int, _int, _int, _int]
    L.oracle_conv2d_i8.restype = _int
    L.oracle_conv2d_i8.argtypes = [_i8p, _i8p, _i8p, _i32p, _i32p, _i32p, _int] + [_int] * 14
    _dp = ctypes.POINTER(ctypes.c_double)
    L.oracle_mpc_forward.restype = None
    L.oracle_mpc_forward.argtypes = [_dp, _dp, _dp, _dp, _dp, _dp, _dp, _int, _int]
    L.oracle_num_threads.restype = _int
    L.oracle_num_threads.argtypes = []
    return L


def _p8(a: np.ndarray):
    assert a.dtype == np.int8 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_i8p)


def _p32(a: Optional[np.ndarray]):
    if a is None:
        return ctypes.cast(None, _i32p)
    assert a.dtype == np.int32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(_i32p)


class Oracle:
    """The oracle's functions bound to one shared object (the default build, or a deliberately
    broken copy that a test compiled to show that the pins notice the breakage)."""

    def __init__(self, so_path: Optional[str] = None):
        self._L = _bind(so_path or build())

    def num_threads(self) -> int:
        return int(self._L.oracle_num_threads())

    def requant(self, acc: int, bias: int, relu: int, mult: int, shift: int):
        """Return (int8 value, overflow flag) of one epilogue evaluation."""
        ovf = _int(0)
        v = self._L.oracle_requant(int(acc), int(bias), int(relu), int(mult), int(shift), ctypes.byref(ovf))
        return int(v), int(ovf.value)

    def requant_fscale(self, acc: int, bias: int, relu: int, scale: float):
        """Return (int8 value, overflow flag) of one float-scale read-out (scale is taken as a binary32 value)."""
        ovf = _int(0)
        v = self._L.oracle_requant_fscale(int(acc), int(bias), int(relu), ctypes.c_float(scale), ctypes.byref(ovf))
        return int(v), int(ovf.value)

    def gemm_i8_fscale(self, A, a_rs, a_cs, B, b_rs, b_cs, ldc, bias, scale, per_channel, M, N, K, relu):
        """C as an (M, ldc) int8 array; scale: float32 array of 1 or N entries."""
        assert scale.dtype == np.float32 and scale.flags["C_CONTIGUOUS"]
        C = np.zeros((M, ldc), dtype=np.int8)
        self._L.oracle_gemm_i8_fscale(_p8(A), a_rs, a_cs, _p8(B), b_rs, b_cs, _p8(C), ldc, _p32(bias),
                                      scale.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), per_channel, M, N, K, relu)
        return C

    def gemm_acc(self, A, a_rs, a_cs, B, b_rs, b_cs, M, N, K) -> np.ndarray:
        acc = np.empty((M, N), dtype=np.int64)
        self._L.oracle_gemm_acc(_p8(A), a_rs, a_cs, _p8(B), b_rs, b_cs, acc.ctypes.data_as(_i64p), M, N, K)
        return acc

    def gemm_i8(self, A, a_rs, a_cs, B, b_rs, b_cs, ldc, bias, mult, shift, per_channel, M, N, K, relu,
                return_overflow: bool = False):
        """C as an (M, ldc) int8 array (columns >= N are left zero)."""
        C = np.zeros((M, ldc), dtype=np.int8)
        ovf = self._L.oracle_gemm_i8(_p8(A), a_rs, a_cs, _p8(B), b_rs, b_cs, _p8(C), ldc,
                                     _p32(bias), _p32(mult), _p32(shift), per_channel, M, N, K, relu)
        return (C, int(ovf)) if return_overflow else C

    def batched_gemm_i8(self, A, a_rs, a_cs, a_bs, B, b_rs, b_cs, b_bs, ldc, c_bs, bias, bias_bs, mult,
                        shift, per_channel, batch, M, N, K, relu, return_overflow: bool = False):
        """C as a flat int8 array of batch*c_bs elements."""
        C = np.zeros(batch * c_bs, dtype=np.int8)
        ovf = self._L.oracle_batched_gemm_i8(_p8(A), a_rs, a_cs, a_bs, _p8(B), b_rs, b_cs, b_bs,
                                             _p8(C), ldc, c_bs, _p32(bias), bias_bs, _p32(mult),
                                             _p32(shift), per_channel, batch, M, N, K, relu)
        return (C, int(ovf)) if return_overflow else C

    def conv2d_i8(self, x, w, bias, mult, shift, per_channel, N, H, W, C, K, R, S, stride_h, stride_w,
                  pad_h, pad_w, relu, n_begin: int = 0, n_end: Optional[int] = None,
                  return_overflow: bool = False):
        """y[N,P,Q,K] int8; only images n_begin <= n < n_end are written (others stay zero)."""
        P = (H + 2 * pad_h - R) // stride_h + 1
        Q = (W + 2 * pad_w - S) // stride_w + 1
        if n_end is None:
            n_end = N
        y = np.zeros((N, P, Q, K), dtype=np.int8)
        ovf = self._L.oracle_conv2d_i8(_p8(x), _p8(w), _p8(y), _p32(bias), _p32(mult), _p32(shift),
                                       per_channel, N, H, W, C, K, R, S, stride_h, stride_w, pad_h,
                                       pad_w, relu, n_begin, n_end)
        return (y, int(ovf)) if return_overflow else y


def _pd(a: Optional[np.ndarray]):
    if a is None:
        return ctypes.cast(None, ctypes.POINTER(ctypes.c_double))
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _mpc_forward(self, Adyn, Bdyn, Kinf, x0, d, return_states: bool = False):
    """u[batch, nhorizon, 4] (and x[batch, nhorizon, 12]) of the TinyMPC forward pass, evaluated in float64."""
    f = lambda a: np.ascontiguousarray(a, dtype=np.float64)
    Adyn, Bdyn, Kinf, x0, d = f(Adyn), f(Bdyn), f(Kinf), f(x0), f(d)
    batch, nh = d.shape[0], d.shape[1]
    assert Adyn.shape == (12, 12) and Bdyn.shape == (12, 4) and Kinf.shape == (4, 12) and x0.shape == (batch, 12) and d.shape[2] == 4
    u = np.zeros((batch, nh, 4), dtype=np.float64)
    xs = np.zeros((batch, nh, 12), dtype=np.float64) if return_states else None
    self._L.oracle_mpc_forward(_pd(Adyn), _pd(Bdyn), _pd(Kinf), _pd(x0), _pd(d), _pd(u), _pd(xs), batch, nh)
    return (u, xs) if return_states else u


Oracle.mpc_forward = _mpc_forward

_default: Optional[Oracle] = None


def lib() -> Oracle:
    """The default oracle (built on first use)."""
    global _default
    if _default is None:
        _default = Oracle()
    return _default


def num_threads() -> int:
    return lib().num_threads()


def requant(*a, **k):
    return lib().requant(*a, **k)


def gemm_acc(*a, **k):
    return lib().gemm_acc(*a, **k)


def requant_fscale(*a, **k):
    return lib().requant_fscale(*a, **k)


def gemm_i8_fscale(*a, **k):
    return lib().gemm_i8_fscale(*a, **k)


def gemm_i8(*a, **k):
    return lib().gemm_i8(*a, **k)


def batched_gemm_i8(*a, **k):
    return lib().batched_gemm_i8(*a, **k)


def conv2d_i8(*a, **k):
    return lib().conv2d_i8(*a, **k)


def mpc_forward(*a, **k):
    return lib().mpc_forward(*a, **k)
