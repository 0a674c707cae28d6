// Generic kernels: one thread per output element, plain loops, any strides and alignments.
// They serve operands the tensor paths cannot take (misaligned, MN-contiguous in unsupported
// combinations, K == 0) and tiny problems, and double as an in-library cross-check of the tensor paths.
#pragma once
#include "epilogue.cuh"
#include "ptx.cuh"

namespace i8 {

struct GenericGemmParams {
    const int8_t* A; int64_t a_rs, a_cs, a_bs;
    const int8_t* B; int64_t b_rs, b_cs, b_bs;
    int8_t* C; int64_t ldc, c_bs;
    const int32_t* bias; int64_t bias_bs;
    const int32_t* mult; const int32_t* shift;
    int per_channel, relu;
    int batch, M, N, K;
    int32_t* D; int64_t ldd; int raw, accumulate;   // raw read-out of the accumulators (see gemm_i8_raw)
    const float* fscale;                            // non-NULL: float-scale read-out (see gemm_i8_fscale)
};

__global__ void __launch_bounds__(256) gemm_i8_generic_kernel(const GenericGemmParams p) {
    const int64_t total = (int64_t)p.batch * p.M * p.N;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(idx % p.N);
        const int64_t rest = idx / p.N;
        const int m = (int)(rest % p.M);
        const int64_t b = rest / p.M;
        const int8_t* a = p.A + b * p.a_bs + (int64_t)m * p.a_rs;
        const int8_t* bb = p.B + b * p.b_bs + (int64_t)n * p.b_cs;
        int32_t acc = 0;
        for (int k = 0; k < p.K; k++) acc += (int32_t)a[(int64_t)k * p.a_cs] * (int32_t)bb[(int64_t)k * p.b_rs];
        if (p.raw) {
            int32_t* dst = p.D + (int64_t)m * p.ldd + n;
            *dst = p.accumulate ? *dst + acc : acc;
            continue;
        }
        const int32_t bias = p.bias ? p.bias[b * p.bias_bs + n] : 0;
        const int ci = p.per_channel ? n : 0;
        if (p.fscale) {
            const int32_t r = requant_fscale(acc, bias, p.relu, p.fscale[ci]);
            p.C[b * p.c_bs + (int64_t)m * p.ldc + n] = (int8_t)min(127, max(-128, r));
            continue;
        }
        p.C[b * p.c_bs + (int64_t)m * p.ldc + n] = (int8_t)requant_wide(acc, bias, p.relu, p.mult[ci], p.shift[ci]);
    }
}

struct GenericConvParams {
    const int8_t* x; const int8_t* w; int8_t* y;
    const int32_t* bias; const int32_t* mult; const int32_t* shift;
    int per_channel, relu;
    int N, H, W, C, K, R, S, P, Q, stride_h, stride_w, pad_h, pad_w;
};

__global__ void __launch_bounds__(256) conv2d_i8_generic_kernel(const GenericConvParams p) {
    const int64_t total = (int64_t)p.N * p.P * p.Q * p.K;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int k = (int)(idx % p.K);
        int64_t rest = idx / p.K;
        const int q = (int)(rest % p.Q); rest /= p.Q;
        const int pp = (int)(rest % p.P);
        const int n = (int)(rest / p.P);
        int32_t acc = 0;
        for (int r = 0; r < p.R; r++) {
            const int h = pp * p.stride_h - p.pad_h + r;
            if (h < 0 || h >= p.H) continue;
            for (int s = 0; s < p.S; s++) {
                const int ww = q * p.stride_w - p.pad_w + s;
                if (ww < 0 || ww >= p.W) continue;
                const int8_t* xp = p.x + (((int64_t)n * p.H + h) * p.W + ww) * p.C;
                const int8_t* wp = p.w + (((int64_t)k * p.R + r) * p.S + s) * p.C;
                for (int c = 0; c < p.C; c++) acc += (int32_t)xp[c] * (int32_t)wp[c];
            }
        }
        const int ci = p.per_channel ? k : 0;
        p.y[idx] = (int8_t)requant_wide(acc, p.bias ? p.bias[k] : 0, p.relu, p.mult[ci], p.shift[ci]);
    }
}

// Unfolds NHWC activations into the row-major matrix [N*P*Q][R*S*C] of the convolution's GEMM form (the column order
// (r, s, c) of the KRSC filters), zeros where a tap falls into the padding.  One 16-byte piece per thread and step
// (C % 16 == 0).  Used for the layers the im2col tensor maps do not take; the product then runs on the tensor path.
struct UnfoldParams {
    const int8_t* x; int8_t* a;
    int N, H, W, C, R, S, P, Q, stride_h, stride_w, pad_h, pad_w;
};

__global__ void __launch_bounds__(256) conv_unfold_i8_kernel(const UnfoldParams p) {
    const int c16 = p.C >> 4;
    const int64_t total = (int64_t)p.N * p.P * p.Q * p.R * p.S * c16;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(idx % c16);
        int64_t rest = idx / c16;
        const int s = (int)(rest % p.S); rest /= p.S;
        const int r = (int)(rest % p.R); rest /= p.R;
        const int q = (int)(rest % p.Q); rest /= p.Q;
        const int pp = (int)(rest % p.P);
        const int n = (int)(rest / p.P);
        const int h = pp * p.stride_h - p.pad_h + r, ww = q * p.stride_w - p.pad_w + s;
        int4 v = make_int4(0, 0, 0, 0);
        if (h >= 0 && h < p.H && ww >= 0 && ww < p.W)
            v = __ldg(reinterpret_cast<const int4*>(p.x + (((int64_t)n * p.H + h) * p.W + ww) * p.C) + c);
        reinterpret_cast<int4*>(p.a)[idx] = v;     // idx is exactly the piece's position in the unfolded matrix
    }
}

// The same for any channel count: the matrix rows are padded with zeros to `kp` (a multiple of 16) bytes, one 16-byte
// piece per thread and step, every byte placed on its own.
struct UnfoldBytesParams {
    const int8_t* x; int8_t* a;
    int N, H, W, C, R, S, P, Q, stride_h, stride_w, pad_h, pad_w;
    int kp;
};

__global__ void __launch_bounds__(256) conv_unfold_bytes_i8_kernel(const UnfoldBytesParams p) {
    const int per_row = p.kp >> 4, K = p.R * p.S * p.C;
    const int64_t total = (int64_t)p.N * p.P * p.Q * per_row;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int piece = (int)(idx % per_row);
        int64_t rest = idx / per_row;
        const int q = (int)(rest % p.Q); rest /= p.Q;
        const int pp = (int)(rest % p.P);
        const int n = (int)(rest / p.P);
        uint32_t w4[4] = {0, 0, 0, 0};
#pragma unroll
        for (int j = 0; j < 16; j++) {
            const int k = piece * 16 + j;
            int8_t v = 0;
            if (k < K) {
                const int c = k % p.C, rs = k / p.C, s = rs % p.S, r = rs / p.S;
                const int h = pp * p.stride_h - p.pad_h + r, ww = q * p.stride_w - p.pad_w + s;
                if (h >= 0 && h < p.H && ww >= 0 && ww < p.W) v = p.x[(((int64_t)n * p.H + h) * p.W + ww) * p.C + c];
            }
            w4[j >> 2] |= (uint32_t)(uint8_t)v << (8 * (j & 3));
        }
        reinterpret_cast<int4*>(p.a)[idx] = make_int4((int)w4[0], (int)w4[1], (int)w4[2], (int)w4[3]);
    }
}

// Copies a strided int8 matrix (element (r, k) at src[r * rs + k * cs]) into a K-contiguous one with rows of `kp` bytes
// (a multiple of 16, zero-padded beyond K): the layout the tensor path wants, for operands whose bases or leading
// dimensions are not multiples of 16 bytes or whose strides are general.
struct PackParams {
    const int8_t* src; int8_t* dst;
    int64_t rs, cs;
    int rows, K, kp;
};

__global__ void __launch_bounds__(256) pack_rows_i8_kernel(const PackParams p) {
    const int per_row = p.kp >> 4;
    const int64_t total = (int64_t)p.rows * per_row;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int piece = (int)(idx % per_row);
        const int64_t r = idx / per_row;
        const int8_t* row = p.src + r * p.rs;
        uint32_t w4[4] = {0, 0, 0, 0};
#pragma unroll
        for (int j = 0; j < 16; j++) {
            const int k = piece * 16 + j;
            const int8_t v = k < p.K ? row[(int64_t)k * p.cs] : (int8_t)0;
            w4[j >> 2] |= (uint32_t)(uint8_t)v << (8 * (j & 3));
        }
        reinterpret_cast<int4*>(p.dst)[idx] = make_int4((int)w4[0], (int)w4[1], (int)w4[2], (int)w4[3]);
    }
}

// Self-test of the bounded wait: one CTA waits on an mbarrier that nothing ever signals.  The wait must give
// up after `limit_cycles`, record DEV_TIMEOUT_TEST in the status word and return normally.
__global__ void bounded_wait_selftest_kernel(long long limit_cycles, unsigned* dev_status) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int stop;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        stop = 0;
        fence_barrier_init();
    }
    __syncthreads();
    const WaitEnv env{&stop, dev_status, limit_cycles};
    mbar_wait_warp(b, 0, env, DEV_TIMEOUT_TEST);
    __syncthreads();
    if (threadIdx.x == 0) mbar_inval(b);
}

}  // namespace i8
