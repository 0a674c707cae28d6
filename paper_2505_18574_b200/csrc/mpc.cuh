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
// the fp32 pipe time within 10 % of each other on B200.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "ptx.cuh"

namespace i8 {

constexpr int MPC_NX = 12, MPC_NU = 4;

// The matrices as the kernel reads them: column-major, so that two neighbouring output rows of one column, (M[r][c],
// M[r+1][c]) with r even, are one aligned 8-byte word, and Kinf negated (u = (-Kinf) x - d).
struct MpcMatrices {
    float At[MPC_NX][MPC_NX];     // At[c][r] = Adyn[r][c]
    float Bt[MPC_NU][MPC_NX];     // Bt[c][r] = Bdyn[r][c]
    float Kt[MPC_NX][MPC_NU];     // Kt[c][r] = -Kinf[r][c]
};

// Packed single precision: one instruction works on two floats held in a 64-bit register (both halves rounded to
// nearest as the scalar instruction would).
__device__ __forceinline__ uint64_t f32x2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f32x2_unpack(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f32x2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t f32x2_mul(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// The two equations for one instance whose x[0] is in `x`; d(i) and put_u(i, ...) abstract where the step vectors live.
// Two output rows share one packed instruction: their coefficients of column c are one 8-byte word of the column-major
// matrix, the other operand is x[c] (or u[c]) in both halves.  That halves the fp32 instruction count (120 packed
// multiply-adds and 16 register copies per step instead of 240 scalar multiply-adds), which is what moves the kernel
// from the fp32 issue rate towards the HBM roof.  The step loop is deliberately not unrolled: each step then reads the
// coefficients from the constant bank instead of pinning all 240 in registers.
template <typename GetD, typename PutU>
__device__ __forceinline__ void mpc_steps(const MpcMatrices& m, float (&x)[MPC_NX], int nhorizon, float4* __restrict__ xs_row,
                                          GetD get_d, PutU put_u) {
#pragma unroll 1
    for (int i = 0; i < nhorizon; i++) {
        const float4 dv = get_d(i);
        if (xs_row) {
#pragma unroll
            for (int q = 0; q < 3; q++) xs_row[i * 3 + q] = make_float4(x[4 * q], x[4 * q + 1], x[4 * q + 2], x[4 * q + 3]);
        }
        uint64_t xd[MPC_NX];
#pragma unroll
        for (int c = 0; c < MPC_NX; c++) xd[c] = f32x2_pack(x[c], x[c]);
        // u = (-Kinf) x - d
        uint64_t u2[MPC_NU / 2] = {f32x2_pack(-dv.x, -dv.y), f32x2_pack(-dv.z, -dv.w)};
#pragma unroll
        for (int c = 0; c < MPC_NX; c++)
#pragma unroll
            for (int rp = 0; rp < MPC_NU / 2; rp++)
                u2[rp] = f32x2_fma(*reinterpret_cast<const uint64_t*>(&m.Kt[c][2 * rp]), xd[c], u2[rp]);
        float ui[MPC_NU];
        f32x2_unpack(u2[0], ui[0], ui[1]);
        f32x2_unpack(u2[1], ui[2], ui[3]);
        put_u(i, make_float4(ui[0], ui[1], ui[2], ui[3]));
        if (i + 1 < nhorizon) {
            uint64_t ud[MPC_NU];
#pragma unroll
            for (int c = 0; c < MPC_NU; c++) ud[c] = f32x2_pack(ui[c], ui[c]);
            uint64_t xn[MPC_NX / 2];
#pragma unroll
            for (int rp = 0; rp < MPC_NX / 2; rp++)
                xn[rp] = f32x2_mul(*reinterpret_cast<const uint64_t*>(&m.At[0][2 * rp]), xd[0]);
#pragma unroll
            for (int c = 1; c < MPC_NX; c++)
#pragma unroll
                for (int rp = 0; rp < MPC_NX / 2; rp++)
                    xn[rp] = f32x2_fma(*reinterpret_cast<const uint64_t*>(&m.At[c][2 * rp]), xd[c], xn[rp]);
#pragma unroll
            for (int c = 0; c < MPC_NU; c++)
#pragma unroll
                for (int rp = 0; rp < MPC_NX / 2; rp++)
                    xn[rp] = f32x2_fma(*reinterpret_cast<const uint64_t*>(&m.Bt[c][2 * rp]), ud[c], xn[rp]);
#pragma unroll
            for (int rp = 0; rp < MPC_NX / 2; rp++) f32x2_unpack(xn[rp], x[2 * rp], x[2 * rp + 1]);
        }
    }
}

// One instance per thread; the next step's d is fetched while the current step computes.  (Staging the 48- and
// 16*nhorizon-byte records through shared memory for coalescing was measured and is no faster.)
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

// Streaming variant (the default when two chunks' records fit in a third of an SM's shared memory): persistent CTAs walk
// chunks of MPC_CHUNK consecutive instances, CTA b taking chunks b, b + gridDim.x, ... so that the CTAs running at any
// moment work on neighbouring memory (whole contiguous ranges per CTA measured 5-40 % slower).  A chunk's x0 and d records
// are two contiguous byte ranges, fetched by one bulk copy each into a ring of `stages` shared-memory slots: a CTA always
// has stages - 1 chunks of loads in flight while it computes, where the one-instance-per-thread loads above keep 16-64
// bytes per thread in flight and stall on them.  Each thread reads its own records from the slot (16-byte accesses; the
// 48- and 80-byte strides are conflict-free per quarter warp) and stores its u vectors to global memory itself (staging
// them in shared memory for a bulk store costs a CTA per SM and measured no faster).
constexpr int MPC_MAX_STAGES = 4;
constexpr unsigned DEV_TIMEOUT_MPC_LOAD = 0x601;    // a chunk's records did not arrive

struct MpcStreamParams {
    const float* x0; const float* d; float* u;
    int batch, nhorizon, stages;
    long long wait_limit_cycles;
    unsigned* dev_status;
};

template <int MPC_CHUNK>
__global__ void __launch_bounds__(MPC_CHUNK)
mpc_forward_stream_kernel(const __grid_constant__ MpcMatrices m, const MpcStreamParams p) {
    extern __shared__ __align__(128) uint8_t mpc_smem[];
    const int nh = p.nhorizon, S = p.stages;
    const uint32_t x_bytes = MPC_CHUNK * MPC_NX * 4, d_bytes = MPC_CHUNK * 16 * nh;     // per full chunk
    const uint32_t in_bytes = x_bytes + d_bytes;
    uint8_t* s_in = mpc_smem;
    uint64_t* s_bar = reinterpret_cast<uint64_t*>(mpc_smem + (size_t)S * in_bytes);
    volatile int* s_stop = reinterpret_cast<volatile int*>(s_bar + MPC_MAX_STAGES);
    const uint32_t bar0 = smem_u32(s_bar);
    const int t = threadIdx.x;
    const int num_chunks = (p.batch + MPC_CHUNK - 1) / MPC_CHUNK;

    if (t == 0) {
        for (int s = 0; s < S; s++) mbar_init(bar0 + 8 * s, 1);
        *s_stop = 0;
        fence_barrier_init();
    }
    __syncthreads();
    const WaitEnv env{s_stop, p.dev_status, p.wait_limit_cycles};

    // thread 0: fetch chunk `c` into slot `s`
    auto fetch = [&](int c, int s) {
        const int count = min(MPC_CHUNK, p.batch - c * MPC_CHUNK);
        const uint32_t xb = (uint32_t)count * MPC_NX * 4, db = (uint32_t)count * 16 * nh;
        const uint32_t dst = smem_u32(s_in + (size_t)s * in_bytes);
        mbar_expect_tx(bar0 + 8 * s, xb + db);
        bulk_load_1d(dst, p.x0 + (size_t)c * MPC_CHUNK * MPC_NX, xb, bar0 + 8 * s);
        bulk_load_1d(dst + x_bytes, p.d + (size_t)c * MPC_CHUNK * 4 * nh, db, bar0 + 8 * s);
    };
    uint32_t armed = 0, armed_phase = 0;             // thread 0: slots with a fetch that may still be in flight
    if (t == 0) {
        for (int s = 0; s < S; s++) {
            const int c = (int)blockIdx.x + s * (int)gridDim.x;
            if (c < num_chunks) { fetch(c, s); armed |= 1u << s; }
        }
    }

    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int c = blockIdx.x; c < num_chunks; c += gridDim.x) {
        ok = mbar_wait(bar0 + 8 * stage, phase, env, DEV_TIMEOUT_MPC_LOAD);
        if (!__syncthreads_and(ok)) { ok = false; break; }      // everybody leaves together when a wait gave up
        if (t == 0) armed &= ~(1u << stage);
        const int count = min(MPC_CHUNK, p.batch - c * MPC_CHUNK);
        const uint8_t* in = s_in + (size_t)stage * in_bytes;
        if (t < count) {
            float x[MPC_NX];
            const float4* xr = reinterpret_cast<const float4*>(in) + t * 3;
#pragma unroll
            for (int q = 0; q < 3; q++) {
                const float4 v = xr[q];
                x[4 * q] = v.x; x[4 * q + 1] = v.y; x[4 * q + 2] = v.z; x[4 * q + 3] = v.w;
            }
            const float4* dr = reinterpret_cast<const float4*>(in + x_bytes) + (size_t)t * nh;
            float4* ug = reinterpret_cast<float4*>(p.u) + ((size_t)c * MPC_CHUNK + t) * nh;
            mpc_steps(m, x, nh, nullptr, [&](int i) { return dr[i]; }, [&](int i, float4 v) { ug[i] = v; });
        }
        __syncthreads();                             // everybody is done with this slot: refill it
        if (t == 0) {
            const int cn = c + S * (int)gridDim.x;
            if (cn < num_chunks) {
                fetch(cn, stage);
                armed |= 1u << stage;
                armed_phase = (armed_phase & ~(1u << stage)) | ((phase ^ 1u) << stage);
            }
        }
        if (++stage == S) { stage = 0; phase ^= 1; }
    }
    if (t == 0 && !ok) {
        // stopping early: let the copies already started land before the CTA retires
        for (int s = 0; s < S; s++)
            if (armed & (1u << s))
                if (!mbar_wait_drain(bar0 + 8 * s, (armed_phase >> s) & 1u, p.wait_limit_cycles))
                    atomicCAS(p.dev_status, 0u, (unsigned)DEV_TIMEOUT_DRAIN);
    }
}

}  // namespace i8
