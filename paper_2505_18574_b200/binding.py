"""ctypes binding of ``libi8ops.so`` with the same entry-point names as ``include/i8ops.h``.

Only argument marshalling happens here: tensors are torch CUDA tensors (torch is used for device memory
and streams), from which pointers, extents and strides are read and passed to the C ABI.  There is no
fallback: if the library is missing or a call reports an error, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libi8ops.so")
_lib = None

PATH_NONE, PATH_GENERIC, PATH_TENSOR, PATH_SMALL, PATH_TENSOR_2SM, PATH_CONV_SLAB = 0, 1, 2, 3, 4, 5
PATH_CHANNEL_MAJOR, PATH_CHANNEL_MAJOR_2SM = 6, 7

_vp = ctypes.c_void_p
_i64 = ctypes.c_int64
_int = ctypes.c_int

# name -> (restype, argtypes); every symbol that include/i8ops.h declares
SIGNATURES = {
    "gemm_i8": (_int, [_vp, _i64, _i64, _vp, _i64, _i64, _vp, _i64, _vp, _vp, _vp, _int, _int, _int, _int, _int, _vp]),
    "gemm_i8_raw": (_int, [_vp, _i64, _i64, _vp, _i64, _i64, _vp, _i64, _int, _int, _int, _int, _vp]),
    "gemm_i8_fscale": (_int, [_vp, _i64, _i64, _vp, _i64, _i64, _vp, _i64, _vp, _vp, _int, _int, _int, _int, _int, _vp]),
    "batched_gemm_i8": (_int, [_vp, _i64, _i64, _i64, _vp, _i64, _i64, _i64, _vp, _i64, _i64, _vp, _i64, _vp, _vp, _int,
                               _int, _int, _int, _int, _int, _vp]),
    "conv2d_i8": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _int] + [_int] * 12 + [_vp]),
    "gemm_i8_host": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _int, _int, _int, _int, _int, _vp]),
    "gemm_i8_host_noalloc": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _int, _int, _int, _int, _int, _vp]),
    "mpc_forward_f32": (_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _int, _int, _vp]),
    "i8_status_string": (ctypes.c_char_p, [_int]),
    "i8ops_last_device_status": (_int, [_vp]),
    "i8ops_selftest_bounded_wait": (_int, [_int, _vp]),
    "i8ops_plan_gemm": (_int, [_int, _int, _int, _int, _vp]),
    "i8ops_set_class_tile": (_int, [_int, _int]),
    "i8ops_set_class_plan": (_int, [_int] * 8),
    "i8ops_last_plan": (_int, [_vp]),
    "i8ops_tmap_cache_stats": (_int, [_vp, _vp]),
    "i8ops_probe_mma_rate": (_int, [_int, _int, _int, _vp, _vp]),
    "i8ops_last_cuda_error": (_int, []),
    "i8ops_last_path": (_int, []),
    "i8ops_last_conv_unfolded": (_int, []),
    "i8ops_last_gemm_packed": (_int, []),
    "i8ops_set_path": (_int, [_int]),
    "i8ops_set_wait_limit_ms": (None, [_int]),
    "i8ops_version": (_int, []),
}


class I8Error(RuntimeError):
    """A call into libi8ops returned a non-zero status."""

    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: i8_status {status} ({status_string(status)})")


def lib() -> ctypes.CDLL:
    """Load ``libi8ops.so`` (built by ``python -m paper_2505_18574_b200.build``); raise if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2505_18574_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().i8_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise I8Error(status, where)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _gemm_i8_args(A, B, C, bias, mult, shift, per_channel, relu, stream=None):
    M, K = A.shape
    K2, N = B.shape
    assert K == K2 and tuple(C.shape) == (M, N) and (C.stride(1) == 1 or N <= 1)
    return (_ptr(A), A.stride(0), A.stride(1), _ptr(B), B.stride(0), B.stride(1), _ptr(C), C.stride(0),
            _ptr(bias), _ptr(mult), _ptr(shift), int(per_channel), M, N, K, int(relu), _stream_ptr(stream))


def gemm_i8(A, B, C, bias, mult, shift, per_channel: int, relu: int, stream=None) -> None:
    """C = epilogue(A . B).  A: (M, K) int8 view, B: (K, N) int8 view (pass ``Bt.t()`` for a column-major B
    stored as (N, K)), C: (M, N) int8 with unit column stride; bias int32 [N] or None; mult/shift int32 [1] or [N]."""
    _check(lib().gemm_i8(*_gemm_i8_args(A, B, C, bias, mult, shift, per_channel, relu, stream)), "gemm_i8")


def gemm_i8_raw(A, B, D, accumulate: bool = False, stream=None) -> None:
    """D (+)= A . B as int32 accumulators (no epilogue).  A: (M, K), B: (K, N) int8 views, D: (M, N) int32."""
    M, K = A.shape
    K2, N = B.shape
    assert K == K2 and tuple(D.shape) == (M, N) and (D.stride(1) == 1 or N <= 1)
    st = lib().gemm_i8_raw(_ptr(A), A.stride(0), A.stride(1), _ptr(B), B.stride(0), B.stride(1), _ptr(D), D.stride(0),
                           int(bool(accumulate)), M, N, K, _stream_ptr(stream))
    _check(st, "gemm_i8_raw")


def gemm_i8_fscale(A, B, C, bias, scale, per_channel: int, relu: int, stream=None) -> None:
    """C = float-scale read-out of A . B (see ``gemm_i8_fscale`` in i8ops.h); scale: float32 CUDA tensor, [1] or [N]."""
    M, K = A.shape
    K2, N = B.shape
    assert K == K2 and tuple(C.shape) == (M, N) and (C.stride(1) == 1 or N <= 1)
    st = lib().gemm_i8_fscale(_ptr(A), A.stride(0), A.stride(1), _ptr(B), B.stride(0), B.stride(1), _ptr(C), C.stride(0),
                              _ptr(bias), _ptr(scale), int(per_channel), M, N, K, int(relu), _stream_ptr(stream))
    _check(st, "gemm_i8_fscale")


def _batched_gemm_i8_args(A, B, C, bias, mult, shift, per_channel, relu, stream=None):
    batch, M, K = A.shape
    _, K2, N = B.shape
    assert K == K2 and tuple(C.shape) == (batch, M, N) and (C.stride(2) == 1 or N <= 1)
    bias_bs = 0
    if bias is not None and bias.dim() == 2:
        bias_bs = bias.stride(0)
    return (_ptr(A), A.stride(1), A.stride(2), A.stride(0), _ptr(B), B.stride(1), B.stride(2), B.stride(0), _ptr(C),
            C.stride(1), C.stride(0), _ptr(bias), bias_bs, _ptr(mult), _ptr(shift), int(per_channel), batch, M, N, K,
            int(relu), _stream_ptr(stream))


def batched_gemm_i8(A, B, C, bias, mult, shift, per_channel: int, relu: int, stream=None) -> None:
    """A: (batch, M, K), B: (batch, K, N), C: (batch, M, N) int8 views; bias int32 (batch, N), (N,) or None."""
    _check(lib().batched_gemm_i8(*_batched_gemm_i8_args(A, B, C, bias, mult, shift, per_channel, relu, stream)),
           "batched_gemm_i8")


def _conv2d_i8_args(x, w, y, bias, mult, shift, per_channel, relu, stride=(1, 1), pad=(0, 0), stream=None):
    N, H, W, C = x.shape
    K, R, S, C2 = w.shape
    assert C == C2 and x.is_contiguous() and w.is_contiguous() and y.is_contiguous()
    return (_ptr(x), _ptr(w), _ptr(y), _ptr(bias), _ptr(mult), _ptr(shift), int(per_channel), N, H, W, C, K, R, S,
            int(stride[0]), int(stride[1]), int(pad[0]), int(pad[1]), int(relu), _stream_ptr(stream))


def conv2d_i8(x, w, y, bias, mult, shift, per_channel: int, relu: int, stride=(1, 1), pad=(0, 0), stream=None) -> None:
    """x: (N, H, W, C), w: (K, R, S, C), y: (N, P, Q, K), all dense int8."""
    _check(lib().conv2d_i8(*_conv2d_i8_args(x, w, y, bias, mult, shift, per_channel, relu, stride, pad, stream)), "conv2d_i8")


class Prepared:
    """One call into the C ABI with its arguments marshalled ahead of time: ``prepare("gemm_i8", A, B.t(), C, ...)``
    reads pointers, extents and strides from the tensors once; calling the object then only crosses the boundary (what a
    C caller's loop does).  The tensors must stay alive and unmoved, and the stream is the one current at preparation."""

    _ARGS = {"gemm_i8": _gemm_i8_args, "batched_gemm_i8": _batched_gemm_i8_args, "conv2d_i8": _conv2d_i8_args}

    def __init__(self, name: str, *tensors, **kw):
        self.name = name
        self._fn = getattr(lib(), name)
        raw = self._ARGS[name](*tensors, **kw)
        self._args = tuple(t(v) if v is not None else None for t, v in zip(SIGNATURES[name][1], raw))
        self._keep = tensors

    def __call__(self) -> None:
        st = self._fn(*self._args)
        if st:
            raise I8Error(st, self.name)

    def with_stream(self, stream) -> "Prepared":
        """The same call on another stream (the stream is the last argument of every compute entry point)."""
        other = object.__new__(Prepared)
        other.name, other._fn, other._keep = self.name, self._fn, self._keep
        other._args = self._args[:-1] + (_vp(_stream_ptr(stream)),)
        return other


def prepare(name: str, *tensors, **kw) -> Prepared:
    return Prepared(name, *tensors, **kw)


def gemm_i8_host(A, B, C, bias, mult, shift, per_channel: int, relu: int, stream=None) -> None:
    """Host-buffer GEMM: A (M, K), B stored column-major as (N, K), C (M, N), all contiguous host tensors or
    numpy arrays (anything with ``data_ptr()`` or ``ctypes.data``); copies in, computes on the GPU, copies out."""
    def hp(a):
        if a is None:
            return None
        return a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data
    M, K = A.shape
    N = B.shape[0]
    st = lib().gemm_i8_host(hp(A), hp(B), hp(C), hp(bias), hp(mult), hp(shift), int(per_channel), M, N, K, int(relu),
                            _stream_ptr(stream))
    _check(st, "gemm_i8_host")


NOALLOC_MAX_BYTES = 16 * 1024 * 1024


def gemm_i8_host_noalloc(A, B, C, bias, mult, shift, per_channel: int, relu: int, stream=None) -> None:
    """gemm_i8_host for callers that may not allocate device memory: same arguments and results, but the device
    copies live in a fixed 16 MiB array inside the library, so the padded operands, vectors and result together must
    fit in ``NOALLOC_MAX_BYTES`` (status 9 otherwise).  Calls share that array: do not overlap them on one GPU."""
    def hp(a):
        if a is None:
            return None
        return a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data
    M, K = A.shape
    N = B.shape[0]
    st = lib().gemm_i8_host_noalloc(hp(A), hp(B), hp(C), hp(bias), hp(mult), hp(shift), int(per_channel), M, N, K,
                                    int(relu), _stream_ptr(stream))
    _check(st, "gemm_i8_host_noalloc")


def mpc_forward_f32(Adyn, Bdyn, Kinf, x0, d, u, xs=None, stream=None) -> None:
    """TinyMPC forward pass.  Adyn (12,12), Bdyn (12,4), Kinf (4,12): host float32 arrays (numpy or CPU tensors);
    x0 (batch,12), d (batch,nh,4), u (batch,nh,4) and optional xs (batch,nh,12): contiguous CUDA float32 tensors."""
    import numpy as np
    mats = [np.ascontiguousarray(np.asarray(a), dtype=np.float32) for a in (Adyn, Bdyn, Kinf)]
    assert mats[0].shape == (12, 12) and mats[1].shape == (12, 4) and mats[2].shape == (4, 12)
    batch, nh = d.shape[0], d.shape[1]
    assert tuple(x0.shape) == (batch, 12) and tuple(u.shape) == (batch, nh, 4) and x0.is_contiguous() and d.is_contiguous()
    st = lib().mpc_forward_f32(mats[0].ctypes.data, mats[1].ctypes.data, mats[2].ctypes.data, _ptr(x0), _ptr(d), _ptr(u),
                               _ptr(xs), batch, nh, _stream_ptr(stream))
    _check(st, "mpc_forward_f32")


class Plan(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("shape_class", "tile_m", "tile_n", "stages", "cta_group", "raster_group", "sticky",
                                             "m_tiles", "n_tiles", "workers", "waves", "b_resident", "epilogue_warps", "kernel")]


def plan_gemm(M: int, N: int, K: int, sm_count: int = 148) -> dict:
    """The tile plan gemm_i8 would use for this shape (host-side query)."""
    pl = Plan()
    _check(lib().i8ops_plan_gemm(int(M), int(N), int(K), int(sm_count), ctypes.byref(pl)), "i8ops_plan_gemm")
    return {n: getattr(pl, n) for n, _ in Plan._fields_}


def last_plan() -> dict:
    """The plan of this thread's most recent launch of the large-tile tensor kernel."""
    pl = Plan()
    _check(lib().i8ops_last_plan(ctypes.byref(pl)), "i8ops_last_plan")
    return {n: getattr(pl, n) for n, _ in Plan._fields_}


def set_class_tile(shape_class: int, tile_n: int) -> None:
    _check(lib().i8ops_set_class_tile(int(shape_class), int(tile_n)), "i8ops_set_class_tile")


def set_class_plan(shape_class: int, base=(0, 0, 0), tile_n: int = 0, cta_group: int = 0, raster_group: int = 0,
                   sticky: int = -1) -> None:
    """Record a schedule for a shape class (see ``i8ops_set_class_plan``); all defaults forgets the entry."""
    _check(lib().i8ops_set_class_plan(int(shape_class), int(base[0]), int(base[1]), int(base[2]), int(tile_n), int(cta_group),
                                      int(raster_group), int(sticky)), "i8ops_set_class_plan")


def last_conv_unfolded() -> bool:
    """Whether the calling thread's most recent convolution ran as an unfold pass followed by the tensor GEMM."""
    return bool(lib().i8ops_last_conv_unfolded())


def last_gemm_packed() -> bool:
    """Whether the calling thread's most recent gemm_i8 ran on packed copies of operands the tensor path could not fetch in place."""
    return bool(lib().i8ops_last_gemm_packed())


def tmap_cache_stats():
    """(hits, misses) of the calling thread's tensor-map cache."""
    h, m = ctypes.c_uint64(0), ctypes.c_uint64(0)
    _check(lib().i8ops_tmap_cache_stats(ctypes.byref(h), ctypes.byref(m)), "i8ops_tmap_cache_stats")
    return int(h.value), int(m.value)


def probe_mma_rate(tile_n: int = 256, reps: int = 8192, ctas: Optional[int] = None, stream=None) -> dict:
    """Run the tensor-core issue-rate probe on `ctas` SMs (default: all) and return the measured int8 peak:
    ``tops`` (whole chip, from the slowest CTA's wall time), ``cycles_per_mma`` (median over CTAs), ``sm_mhz`` (SM cycles per
    nanosecond during the probe) and ``us`` (duration)."""
    import torch
    if ctas is None:
        ctas = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    out = torch.zeros((ctas, 4), dtype=torch.int64, device="cuda")
    _check(lib().i8ops_probe_mma_rate(int(tile_n), int(reps), int(ctas), _ptr(out), _stream_ptr(stream)), "i8ops_probe_mma_rate")
    torch.cuda.synchronize()
    o = out.cpu().numpy()
    if (o[:, 2] == 0).any():
        raise I8Error(8, "i8ops_probe_mma_rate")
    ns = float(o[:, 2].max())
    ops = float(ctas) * reps * 2.0 * 128 * tile_n * 32
    cyc = sorted(o[:, 1].tolist())[ctas // 2]
    return {"tile_n": tile_n, "reps": reps, "ctas": ctas, "tops": ops / ns / 1e3, "cycles_per_mma": cyc / reps,
            "sm_mhz": cyc / float(sorted(o[:, 2].tolist())[ctas // 2]) * 1e3, "us": ns / 1e3,
            "distinct_sms": int(len(set(o[:, 3].tolist())))}


def last_device_status(stream=None) -> int:
    return lib().i8ops_last_device_status(_stream_ptr(stream))


def last_path() -> int:
    return lib().i8ops_last_path()


def set_path(mode: int) -> int:
    return lib().i8ops_set_path(int(mode))


def set_wait_limit_ms(ms: int) -> None:
    lib().i8ops_set_wait_limit_ms(int(ms))
