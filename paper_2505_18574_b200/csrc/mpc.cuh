// Fine-grained linear algebra as the paper runs it: the forward pass of the TinyMPC primal update
// (Code Examples appendix, "TinyMPC Primal Update Forward Pass"):
//     u[i]   = -Kinf * x[i] - d[i]
//     x[i+1] =  Adyn * x[i] + Bdyn * u[i]          i = 0 .. nhorizon-1, x[nhorizon] not formed
// 12 states, 4 inputs, fp32 as in the paper.  Many independent instances share the three matrices (the
// paper's "hoist the constant matrices out of the loop" step becomes: they travel as a kernel argument and
// are read through the constant bank), one thread carries one instance's state in registers through the
// whole horizon (no round trip through memory between steps, the paper's "keep data resident in the
// accumulator"), and every global access is a 16-byte vector.  Per instance: 48 + 32*nhorizon bytes (x0, d, u; plus
// 48*nhorizon when the states are also written) and 100*nhorizon + 396*(nhorizon-1) flops, which puts the HBM time and
// the fp32 issue time within 10 % of each other on B200.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace i8 {

constexpr int MPC_NX = 12, MPC_NU = 4;

struct MpcMatrices {
    float A[MPC_NX][MPC_NX];
    float B[MPC_NX][MPC_NU];
    float K[MPC_NU][MPC_NX];
};

// The two equations for one instance whose x[0] is in `x`; d(i) and put_u(i, ...) abstract where the step vectors live.
// The step loop is deliberately not unrolled: each step then reads the matrices straight from the constant bank as
// instruction operands instead of pinning all 240 coefficients in registers.
template <typename GetD, typename PutU>
__device__ __forceinline__ void mpc_steps(const MpcMatrices& m, float (&x)[MPC_NX], int nhorizon, float4* __restrict__ xs_row,
                                          GetD get_d, PutU put_u) {
#pragma unroll 1
    for (int i = 0; i < nhorizon; i++) {
        const float4 dv = get_d(i);
        const float di[4] = {dv.x, dv.y, dv.z, dv.w};
        if (xs_row) {
#pragma unroll
            for (int q = 0; q < 3; q++) xs_row[i * 3 + q] = make_float4(x[4 * q], x[4 * q + 1], x[4 * q + 2], x[4 * q + 3]);
        }
        float ui[MPC_NU];
#pragma unroll
        for (int r = 0; r < MPC_NU; r++) {
            float kx = 0.f;
#pragma unroll
            for (int c = 0; c < MPC_NX; c++) kx = fmaf(m.K[r][c], x[c], kx);
            ui[r] = -kx - di[r];
        }
        put_u(i, make_float4(ui[0], ui[1], ui[2], ui[3]));
        if (i + 1 < nhorizon) {
            float xn[MPC_NX];
#pragma unroll
            for (int r = 0; r < MPC_NX; r++) {
                float ax = 0.f, bu = 0.f;
#pragma unroll
                for (int c = 0; c < MPC_NX; c++) ax = fmaf(m.A[r][c], x[c], ax);
#pragma unroll
                for (int c = 0; c < MPC_NU; c++) bu = fmaf(m.B[r][c], ui[c], bu);
                xn[r] = ax + bu;
            }
#pragma unroll
            for (int r = 0; r < MPC_NX; r++) x[r] = xn[r];
        }
    }
}

// One instance per thread; the next step's d is fetched while the current step computes.  (Staging the 48- and
// 16*nhorizon-byte records through shared memory for coalescing was measured and is no faster: with 2084 flops per
// 208 bytes the kernel sits on the fp32 issue rate as much as on HBM.)
__global__ void __launch_bounds__(128, 5)
mpc_forward_f32_kernel(const __grid_constant__ MpcMatrices m, const float4* __restrict__ x0, const float4* __restrict__ d,
                       float4* __restrict__ u, float4* __restrict__ xs, int batch, int nhorizon) {
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < batch; b += (int64_t)gridDim.x * blockDim.x) {
        float x[MPC_NX];
#pragma unroll
        for (int q = 0; q < 3; q++) {
            const float4 v = x0[b * 3 + q];
            x[4 * q] = v.x; x[4 * q + 1] = v.y; x[4 * q + 2] = v.z; x[4 * q + 3] = v.w;
        }
        float4 dnext = d[b * nhorizon];
        mpc_steps(m, x, nhorizon, xs ? xs + b * nhorizon * 3 : nullptr,
                  [&](int i) {
                      const float4 dv = dnext;
                      if (i + 1 < nhorizon) dnext = d[b * nhorizon + i + 1];
                      return dv;
                  },
                  [&](int i, float4 v) { u[b * nhorizon + i] = v; });
    }
}

}  // namespace i8
