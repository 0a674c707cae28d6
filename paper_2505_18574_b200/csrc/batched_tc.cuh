// Small-tile tensor path: many independent products with M, N, K <= 64 (the paper's fine-grained linear
// algebra: low reuse, a high ratio of data movement to computation; Evaluation, "Fine-Grained Linear Algebra").
//
// Two problems share one tcgen05.mma: their A tiles are stacked along M (128 rows) and their B tiles sit side
// by side along N (128 columns), so one 128 x 128 x 32 instruction pair computes the 2 x 2 block matrix
//     [A0; A1] . [B0 | B1]
// of which the diagonal blocks A0.B0 (lanes 0..63, columns 0..63) and A1.B1 (lanes 64..127, columns 64..127)
// are the wanted products; the off-diagonal blocks are never read.  The work is HBM-bound (12 KiB moved per
// 64^3 problem), so spending half of an otherwise idle tensor pipe buys full 128-lane tiles and plain loads.
//
//   warp 0       producer : two 3-D TMA loads per pair (A pair, B pair) into a ring slot, 64-byte swizzle
//   warp 1       MMA      : K/32 instructions per pair into one of ACC tensor-memory accumulators (128 columns each)
//   warps 2..    epilogue : ACC groups of 4 warps; group g serves accumulator g, so up to ACC pairs are read
//                           out concurrently while the MMA warp runs ahead
//
// B may be K-contiguous (column-major) or N-contiguous (row-major); the latter is consumed directly through an
// MN-major shared-memory descriptor, no transpose pass.
#pragma once
#include "epilogue.cuh"
#include "ptx.cuh"

namespace i8 {

constexpr int PAIR_UMMA_K = 32;                     // K per tcgen05.mma for 8-bit operands
constexpr int PAIR_ACC = 4;                         // accumulators = epilogue groups
constexpr int PAIR_STAGES = 4;                      // ring slots (measured: 3 to 5 are equally fast, 8 and 12 slower)
constexpr int PAIR_TILE_BYTES = 2 * 64 * 64;        // one operand of a pair
constexpr int PAIR_THREADS = 64 + 128 * PAIR_ACC;

struct BatchedPairParams {
    int8_t* C;
    int64_t ldc, c_bs;
    const int32_t* bias;
    int64_t bias_bs;
    const int32_t* mult;
    const int32_t* shift;
    int per_channel, relu;
    int batch, M, N, K;
    int b_mn_major;             // B is N-contiguous
    int c_vec_ok;               // C, ldc and c_bs are 16-byte aligned
    int bias_vec_ok;            // bias and bias_bs are 16-byte aligned (int4 loads)
    long long wait_limit_cycles;
    unsigned* dev_status;
};

struct PairSmem {
    static constexpr int OFF_A = 0;
    static constexpr int OFF_B = OFF_A + PAIR_STAGES * PAIR_TILE_BYTES;
    static constexpr int OFF_CONST = OFF_B + PAIR_STAGES * PAIR_TILE_BYTES;   // 6 int32[64] arrays
    static constexpr int OFF_BAR = OFF_CONST + 6 * 64 * 4;                    // full[S], empty[S], acc_full[ACC], acc_empty[ACC]
    static constexpr int OFF_MISC = OFF_BAR + (2 * PAIR_STAGES + 2 * PAIR_ACC) * 8;
    static constexpr int TOTAL = OFF_MISC + 16;
    static constexpr int DYN_BYTES = TOTAL + 1024;
    static constexpr int TMEM_COLS = 128 * PAIR_ACC;                          // 512
};

// 32 consecutive bias entries starting at column n0 (zeros where there is no bias or no such column).
__device__ __forceinline__ void load_bias32(const int32_t* brow, int n0, int N, bool vec_ok, int4 (&bq)[8]) {
#pragma unroll
    for (int j = 0; j < 8; j++) bq[j] = make_int4(0, 0, 0, 0);
    if (!brow) return;
    if (vec_ok && n0 + 32 <= N) {
#pragma unroll
        for (int j = 0; j < 8; j++) bq[j] = __ldg(reinterpret_cast<const int4*>(brow + n0) + j);
    } else {
#pragma unroll
        for (int j = 0; j < 8; j++) {
            const int c = n0 + 4 * j;
            if (c + 0 < N) bq[j].x = __ldg(brow + c + 0);
            if (c + 1 < N) bq[j].y = __ldg(brow + c + 1);
            if (c + 2 < N) bq[j].z = __ldg(brow + c + 2);
            if (c + 3 < N) bq[j].w = __ldg(brow + c + 3);
        }
    }
}

// Epilogue arithmetic of one 32-column chunk.  MODE 0: shift-32 form, one multiplier for all channels;
// MODE 1: shift-32 form, per-channel multipliers from shared memory; MODE 2: window form (any scale).
template <int MODE, bool RELU>
__device__ __forceinline__ void pair_chunk(const int32_t (&v)[32], const int4 (&bq)[8], int n0, int32_t m2_shared,
                                           const int32_t* s_m2, const int32_t* s_lo, const int32_t* s_hi, const int32_t* s_mult,
                                           const int32_t* s_shift, const int32_t* s_rnd, uint32_t (&out)[8]) {
#pragma unroll
    for (int j = 0; j < 8; j++) {
        const int bb[4] = {bq[j].x, bq[j].y, bq[j].z, bq[j].w};
        int32_t r[4];
#pragma unroll
        for (int e = 0; e < 4; e++) {
            const int c = n0 + 4 * j + e;
            if (MODE == 2) {
                r[e] = requant_fast(v[4 * j + e], bb[e], s_lo[c], s_hi[c], s_mult[c], s_shift[c], s_rnd[c]);
            } else {
                // high word of max(acc + bias, 0) * m2 + 2^31
                int32_t tt = v[4 * j + e] + bb[e];
                if (RELU) tt = max(tt, 0);
                const int32_t m2 = MODE == 1 ? s_m2[c] : m2_shared;
                const unsigned long long pr = (unsigned long long)((long long)tt * (long long)m2) + (1ull << 31);
                r[e] = (int32_t)(uint32_t)(pr >> 32);
            }
        }
        out[j] = pack_sat4(r[0], r[1], r[2], r[3]);
    }
}

__global__ void __launch_bounds__(PAIR_THREADS, 1)
batched_pair_i8_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const BatchedPairParams p) {
    using L = PairSmem;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sbase = raw + pad;
    const uint32_t sA = sbase + L::OFF_A, sB = sbase + L::OFF_B;
    int32_t* s_m2 = reinterpret_cast<int32_t*>(smem + L::OFF_CONST);   // shift-32 multipliers
    int32_t* s_lo = s_m2 + 64;
    int32_t* s_hi = s_lo + 64;
    int32_t* s_mult = s_hi + 64;
    int32_t* s_shift = s_mult + 64;
    int32_t* s_rnd = s_shift + 64;
    const uint32_t bar_full = sbase + L::OFF_BAR;
    const uint32_t bar_empty = bar_full + PAIR_STAGES * 8;
    const uint32_t bar_acc_full = bar_empty + PAIR_STAGES * 8;
    const uint32_t bar_acc_empty = bar_acc_full + PAIR_ACC * 8;
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_MISC);
    volatile int* s_stop = reinterpret_cast<volatile int*>(smem + L::OFF_MISC + 4);

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    const WaitEnv env{s_stop, p.dev_status, p.wait_limit_cycles};

    if (threadIdx.x == 0) {
        for (int s = 0; s < PAIR_STAGES; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < PAIR_ACC; b++) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, 128);
        }
        *s_stop = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(s_tmem)), L::TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    grid_launch_dependents();
    grid_dependency_wait();   // global memory is touched from here on
    // per-channel constants of the 64 output columns (shared by every problem of the batch)
    bool my32 = true;
    if (threadIdx.x < 64) {
        const int n = threadIdx.x;
        int32_t mult = 0, shift = 1;
        if (n < p.N) {
            mult = p.mult[p.per_channel ? n : 0];
            shift = p.shift[p.per_channel ? n : 0];
        }
        const ChanConst cc = make_chan_const(mult, shift, p.relu);
        s_lo[n] = cc.lo; s_hi[n] = cc.hi; s_mult[n] = cc.mult; s_shift[n] = cc.shift; s_rnd[n] = cc.rnd;
        // shift-32 form with the bias added explicitly (it differs per problem): needs |scale| < 1/2
        my32 = shift >= 1 && mult >= -(1 << (shift - 1)) && mult < (1 << (shift - 1));
        s_m2[n] = my32 ? (int32_t)((uint32_t)mult << (32 - shift)) : 0;
    }
    tc_fence_before();
    const bool all32 = __syncthreads_and(my32) != 0;
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *s_tmem, 0);

    const int num_pairs = (p.batch + 1) >> 1;
    const int ksteps = (p.K + PAIR_UMMA_K - 1) / PAIR_UMMA_K;      // 1 or 2

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        int stage = 0;
        uint32_t phase = 0, issued = 0, issued_phase = 0;
        for (int t = blockIdx.x; t < num_pairs; t += gridDim.x) {
            if (!mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1, env, DEV_TIMEOUT_PRODUCER)) break;
            const uint32_t full = bar_full + 8 * stage;
            if (elect_one()) {
                mbar_expect_tx(full, 2 * PAIR_TILE_BYTES);
                tma_load_3d(sA + stage * PAIR_TILE_BYTES, &tmA, full, 0, 0, 2 * t);
                tma_load_3d(sB + stage * PAIR_TILE_BYTES, &tmB, full, 0, 0, 2 * t);
            }
            issued |= 1u << stage;
            issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
            if (++stage == PAIR_STAGES) { stage = 0; phase ^= 1; }
        }
        if (*s_stop) {
            for (int s = 0; s < PAIR_STAGES; s++)
                if (issued & (1u << s))
                    if (!mbar_wait_drain(bar_full + 8 * s, (issued_phase >> s) & 1u, p.wait_limit_cycles))
                        atomicCAS(p.dev_status, 0u, (unsigned)DEV_TIMEOUT_DRAIN);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc = make_idesc_i8(128, 128, 0, p.b_mn_major);
        // A: K-major rows of 64 bytes, 64-byte swizzle, 8-row groups 512 bytes apart.
        const uint64_t a_hi = make_smem_desc(0, 16, 512, SWZ_64B);
        // B, K-major: the same.  B, MN-major: 64 bytes of N contiguous per K row, 8 K rows per 512-byte group
        // (stride offset), the second problem's 64 columns one tile (4096 bytes) further (leading offset).
        const uint64_t b_hi = p.b_mn_major ? make_smem_desc(0, 4096, 512, SWZ_64B) : a_hi;
        const uint32_t b_kstep = p.b_mn_major ? 32 * 64 : PAIR_UMMA_K;   // bytes per 32 of K
        int stage = 0, acc = 0;
        uint32_t phase = 0, acc_phase = 0;
        for (int t = blockIdx.x; t < num_pairs; t += gridDim.x) {
            if (!mbar_wait_warp(bar_acc_empty + 8 * acc, acc_phase ^ 1, env, DEV_TIMEOUT_MMA_ACC)) break;
            if (!mbar_wait_warp(bar_full + 8 * stage, phase, env, DEV_TIMEOUT_MMA_FULL)) break;
            tc_fence_after();
            if (elect_one()) {
                const uint32_t a0 = sA + stage * PAIR_TILE_BYTES, b0 = sB + stage * PAIR_TILE_BYTES;
                for (int k = 0; k < ksteps; k++) {
                    const uint64_t ad = a_hi | (uint64_t)(((a0 + k * PAIR_UMMA_K) & 0x3FFFFu) >> 4);
                    const uint64_t bd = b_hi | (uint64_t)(((b0 + k * b_kstep) & 0x3FFFFu) >> 4);
                    mma_i8_ss(tmem_base + acc * 128, ad, bd, idesc, k != 0 ? 1u : 0u);
                }
                tc_commit(bar_empty + 8 * stage);
                tc_commit(bar_acc_full + 8 * acc);
            }
            __syncwarp();
            if (++stage == PAIR_STAGES) { stage = 0; phase ^= 1; }
            if (++acc == PAIR_ACC) { acc = 0; acc_phase ^= 1; }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue: group g owns accumulator g
        const int g = (warp - 2) >> 2;
        const int quarter = warp & 3;
        const int which = quarter >> 1;                    // problem of the pair held by this lane quarter
        const int row = (quarter & 1) * 32 + lane;         // row inside that problem
        const int32_t m2_shared = s_m2[0];
        uint32_t acc_phase = 0;
        int seq = 0;                                       // index of this CTA's pair, to pick every PAIR_ACC-th one
        for (int t = blockIdx.x; t < num_pairs; t += gridDim.x, seq++) {
            if ((seq % PAIR_ACC) != g) continue;
            const int prob = 2 * t + which;
            const bool live = prob < p.batch && row < p.M;
            int8_t* crow = p.C + (int64_t)prob * p.c_bs + (int64_t)row * p.ldc;
            const int32_t* brow = (p.bias && prob < p.batch) ? p.bias + (int64_t)prob * p.bias_bs : nullptr;
            // the bias of the first 32 columns does not depend on the product: fetch it before waiting
            int4 bq[8];
            load_bias32(brow, 0, p.N, p.bias_vec_ok != 0, bq);
            bool ok = mbar_wait(bar_acc_full + 8 * g, acc_phase, env, DEV_TIMEOUT_EPILOGUE);
            ok = named_barrier_and(1 + g, 128, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t0 = tmem_base + g * 128 + which * 64 + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
            for (int ch = 0; ch < 2; ch++) {
                const int n0 = 32 * ch;
                if (n0 >= p.N) break;
                int32_t v[32];
                tmem_ld_32x32(t0 + n0, v);
                tmem_ld_wait();
                uint32_t out[8];
                if (all32) {
                    if (p.per_channel) {
                        if (p.relu) pair_chunk<1, true>(v, bq, n0, m2_shared, s_m2, s_lo, s_hi, s_mult, s_shift, s_rnd, out);
                        else pair_chunk<1, false>(v, bq, n0, m2_shared, s_m2, s_lo, s_hi, s_mult, s_shift, s_rnd, out);
                    } else {
                        if (p.relu) pair_chunk<0, true>(v, bq, n0, m2_shared, s_m2, s_lo, s_hi, s_mult, s_shift, s_rnd, out);
                        else pair_chunk<0, false>(v, bq, n0, m2_shared, s_m2, s_lo, s_hi, s_mult, s_shift, s_rnd, out);
                    }
                } else {
                    pair_chunk<2, false>(v, bq, n0, m2_shared, s_m2, s_lo, s_hi, s_mult, s_shift, s_rnd, out);
                }
                if (ch == 0 && p.N > 32) load_bias32(brow, 32, p.N, p.bias_vec_ok != 0, bq);   // next chunk's bias, in flight during the stores
                if (live) {
                    if (p.c_vec_ok && n0 + 32 <= p.N) {
                        uint4* dst = reinterpret_cast<uint4*>(crow + n0);
                        dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
                        dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; j++)
                            if (n0 + j < p.N) crow[n0 + j] = (int8_t)((out[j >> 2] >> (8 * (j & 3))) & 0xff);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar_acc_empty + 8 * g);
            acc_phase ^= 1;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, L::TMEM_COLS);
    }
}

}  // namespace i8
