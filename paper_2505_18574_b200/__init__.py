"""i8ops for B200: int8 GEMM / conv2d / batched GEMM with a fused requantising epilogue.

``binding`` holds the ctypes front end of the C-ABI library ``libi8ops.so`` (argument marshalling only:
every step of the computation runs in the CUDA kernels).  ``inputs`` holds the seeded synthetic workloads.
``build`` compiles the library with nvcc for sm_100a.
"""
from .binding import (I8Error, batched_gemm_i8, conv2d_i8, gemm_i8, gemm_i8_fscale, gemm_i8_host, gemm_i8_host_noalloc, gemm_i8_raw, last_device_status, last_path, last_conv_unfolded, last_gemm_packed, mpc_forward_f32,
                      lib, plan_gemm, last_plan, prepare, probe_mma_rate, set_class_plan, set_class_tile, tmap_cache_stats, set_path, set_wait_limit_ms, status_string, PATH_GENERIC, PATH_NONE, PATH_SMALL,
                      PATH_TENSOR, PATH_TENSOR_2SM, PATH_CONV_SLAB, PATH_CHANNEL_MAJOR, PATH_CHANNEL_MAJOR_2SM)

__all__ = ["I8Error", "batched_gemm_i8", "conv2d_i8", "gemm_i8", "gemm_i8_fscale", "gemm_i8_host", "gemm_i8_host_noalloc", "gemm_i8_raw", "last_device_status", "last_path", "last_conv_unfolded", "last_gemm_packed", "mpc_forward_f32",
           "lib", "plan_gemm", "last_plan", "prepare", "probe_mma_rate", "set_class_plan", "set_class_tile", "tmap_cache_stats", "set_path", "set_wait_limit_ms", "status_string", "PATH_GENERIC", "PATH_NONE", "PATH_SMALL",
           "PATH_TENSOR", "PATH_TENSOR_2SM", "PATH_CONV_SLAB", "PATH_CHANNEL_MAJOR", "PATH_CHANNEL_MAJOR_2SM"]
