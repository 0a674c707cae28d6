"""CPU oracle (test infrastructure).  Only the tests, the smoke check and the benchmark's
CPU-baseline / reference legs may import this package; the CUDA path never does."""
from .cpu_oracle import (Oracle, build, lib, requant, requant_fscale, gemm_acc, gemm_i8, gemm_i8_fscale, batched_gemm_i8, conv2d_i8,
                         mpc_forward, num_threads)

__all__ = ["Oracle", "build", "lib", "requant", "requant_fscale", "gemm_acc", "gemm_i8", "gemm_i8_fscale", "batched_gemm_i8", "conv2d_i8", "mpc_forward",
           "num_threads"]
