// Channel-major tensor path: the product is computed transposed, output channels on the tensor-memory lanes.
//
// tcgen05.mma fixes its M extent at 128 (256 for a CTA pair) but lets N be any multiple of 16 up to 256.  The large-
// tile kernel puts output rows (pixels) on M and channels on N; this kernel swaps the roles:
//     D^T[channel][pixel] = sum_k W[channel][k] * X[pixel][k]
// with a block of 128 (one CTA) or 256 (a CTA pair, cta_group::2) output channels on the lanes and a strip of `pw`
// output rows / pixels on the columns, pw chosen by the host per problem.  Two things follow:
//   * the strip width is a free parameter in steps of 16, so the number of tiles can be matched to the number of SMs
//     (a layer with 12544 pixels and 256 filters gives 49 tiles of 256 x 256, two thirds of the chip's 74 CTA pairs; with
//     pw = 176 it gives 72);
//   * every epilogue thread owns ONE output channel, so bias, multiplier and shift are three registers loaded once per
//     channel block instead of shared-memory broadcasts per output (which, through the load/store pipe that also feeds
//     the tensor core its operands, bounded the read-out of the large-tile kernel at about 2 us per 128 x 256 tile).
// The price is a transpose on the way out: a thread holds 32 pixels of one channel, the output wants the channels of
// one pixel side by side.  Four neighbouring lanes (four channels) exchange their packed bytes in two shuffle rounds so
// that every lane ends up with words of "4 channels x 1 pixel"; one store instruction of the warp then writes four
// pixels' 32-byte channel segments, each a full memory sector.  (Measured alternatives: byte stores into a shared-memory
// staging tile cost 2 us per exposed tile (four lanes writing different bytes of one word serialise), and handing the
// staged tile to the TMA engine in 16-pixel boxes another 1 us.)
//
// Roles, ring, barriers and bounded waits are those of gemm_tc.cuh.  Operand names below follow the instruction, not
// the caller's matrices: the "A side" (128 rows per CTA) holds weights / the caller's B, the "B side" (pw rows, half
// per CTA in a pair) holds activations / the caller's A, fetched by im2col loads for convolutions.
#pragma once
#include "gemm_tc.cuh"

namespace i8 {

constexpr int SWAP_MAX_STAGES = 8;
#ifndef SWAP_EPI_WARPS_N
#define SWAP_EPI_WARPS_N 8
#endif
constexpr int SWAP_EPI_WARPS = SWAP_EPI_WARPS_N;      // a multiple of 4: warps sharing a lane quarter split the strip's columns
constexpr int SWAP_UNIT = 16;                         // granularity of the strip width (tcgen05.mma: N is a multiple of 16)

struct SwapParams {
    int8_t* C;                  // [M][ldc], row-major: rows are pixels / the caller's M, columns are channels / its N
    int64_t ldc;
    const int32_t* bias;
    const int32_t* mult;
    const int32_t* shift;
    const float* fscale;        // non-NULL: float-scale read-out (one entry or N), mult / shift unused
    int per_channel, relu;
    int M, N, K;
    int pw;                     // strip width: rows of C per tile, a multiple of 16, at most 256
    int b_rows;                 // rows of the strip one CTA loads: pw (one CTA) or pw / 2 (pair)
    int c_word_ok;              // C and ldc are 4-byte aligned and N is a multiple of 4: channel quads go out as 32-bit stores
    int m_tiles, n_blocks, num_tiles;
    uint32_t inv_nb;            // floor(2^32 / n_blocks) (0xffffffff for 1)
    int stages;                 // ring slots in use (2 .. SWAP_MAX_STAGES)
    int b_stage_bytes;          // b_rows * 128
    int tmem_cols;              // power of two >= 2 * pw, >= 32
    int off_b, off_bar;         // shared-memory offsets from the 1024-byte aligned base
    KLoop kl;
    long long wait_limit_cycles;
    unsigned* dev_status;
};

// Per-thread epilogue constants of one output channel.
struct SwapChan {
    int32_t bias, m2;
    long long c64;
    ChanConst cc;
    float fscale;
    int form;                   // 0 folded shift-32 form, 1 shift-32 form with ReLU ahead of the scale, 2 window form, 3 float scale
};

__device__ __forceinline__ SwapChan make_swap_chan(int32_t bias, int32_t mult, int32_t shift, int relu) {
    SwapChan c;
    c.bias = bias;
    const bool ok32 = make_shift32_mult(mult, shift, c.m2);
    c.c64 = make_fold_addend(bias, c.m2);
    c.cc = make_chan_const(mult, shift, relu);
    c.form = ok32 ? ((!relu || c.m2 >= 0) ? 0 : 1) : 2;
    c.fscale = 0.f;
    return c;
}

// Requantise `count` (16 or 32) accumulators of one channel and pack them four to a word.
// `all_fold`: every lane of the warp is in the folded form (the common case: positive scales below one half), known
// warp-uniformly, so that the hot path is straight-line code without a per-lane branch.
template <int COUNT>
__device__ __forceinline__ void swap_requant(const int32_t (&v)[32], const SwapChan& ch, int relu, bool all_fold, uint32_t (&out)[8]) {
    if (all_fold) {
        if (relu) {
#pragma unroll
            for (int j = 0; j < COUNT / 4; j++)
                out[j] = relu_s8x4(pack_sat4(requant_fold(v[4 * j + 0], ch.m2, ch.c64), requant_fold(v[4 * j + 1], ch.m2, ch.c64),
                                             requant_fold(v[4 * j + 2], ch.m2, ch.c64), requant_fold(v[4 * j + 3], ch.m2, ch.c64)));
        } else {
#pragma unroll
            for (int j = 0; j < COUNT / 4; j++)
                out[j] = pack_sat4(requant_fold(v[4 * j + 0], ch.m2, ch.c64), requant_fold(v[4 * j + 1], ch.m2, ch.c64),
                                   requant_fold(v[4 * j + 2], ch.m2, ch.c64), requant_fold(v[4 * j + 3], ch.m2, ch.c64));
        }
    } else if (ch.form == 0) {
#pragma unroll
        for (int j = 0; j < COUNT / 4; j++) {
            const uint32_t pk = pack_sat4(requant_fold(v[4 * j + 0], ch.m2, ch.c64), requant_fold(v[4 * j + 1], ch.m2, ch.c64),
                                          requant_fold(v[4 * j + 2], ch.m2, ch.c64), requant_fold(v[4 * j + 3], ch.m2, ch.c64));
            out[j] = relu ? relu_s8x4(pk) : pk;
        }
    } else if (ch.form == 1) {
#pragma unroll
        for (int j = 0; j < COUNT / 4; j++)
            out[j] = pack_sat4(requant_shift32<true>(v[4 * j + 0], ch.bias, ch.m2), requant_shift32<true>(v[4 * j + 1], ch.bias, ch.m2),
                               requant_shift32<true>(v[4 * j + 2], ch.bias, ch.m2), requant_shift32<true>(v[4 * j + 3], ch.bias, ch.m2));
    } else if (ch.form == 3) {
#pragma unroll
        for (int j = 0; j < COUNT / 4; j++)
            out[j] = pack_sat4(requant_fscale(v[4 * j + 0], ch.bias, relu, ch.fscale), requant_fscale(v[4 * j + 1], ch.bias, relu, ch.fscale),
                               requant_fscale(v[4 * j + 2], ch.bias, relu, ch.fscale), requant_fscale(v[4 * j + 3], ch.bias, relu, ch.fscale));
    } else {
#pragma unroll
        for (int j = 0; j < COUNT / 4; j++)
            out[j] = pack_sat4(requant_fast(v[4 * j + 0], ch.bias, ch.cc.lo, ch.cc.hi, ch.cc.mult, ch.cc.shift, ch.cc.rnd),
                               requant_fast(v[4 * j + 1], ch.bias, ch.cc.lo, ch.cc.hi, ch.cc.mult, ch.cc.shift, ch.cc.rnd),
                               requant_fast(v[4 * j + 2], ch.bias, ch.cc.lo, ch.cc.hi, ch.cc.mult, ch.cc.shift, ch.cc.rnd),
                               requant_fast(v[4 * j + 3], ch.bias, ch.cc.lo, ch.cc.hi, ch.cc.mult, ch.cc.shift, ch.cc.rnd));
    }
}

// 4 x 4 byte transpose across the four lanes of a quad.  In: word j of lane q*4 + i holds pixels 4j .. 4j+3 of channel
// q*4 + i.  Out: word j of that lane holds channels q*4 .. q*4+3 of pixel 4j + swap_pixel_of_lane(i).  Two rounds: with
// the neighbour (lane ^ 1) bytes are interleaved into (channel pair x pixel pair) words, with lane ^ 2 the 16-bit halves.
// The byte selectors depend only on the lane, so they are registers, not branches.
__device__ __forceinline__ int swap_pixel_of_lane(int lane) { return 2 * (lane & 1) + ((lane >> 1) & 1); }
template <int WORDS>
__device__ __forceinline__ void quad_transpose(uint32_t (&w)[8], int lane) {
    // even lane keeps pixels 0,1: [me.b0, other.b0, me.b1, other.b1]; odd lane keeps pixels 2,3: [other.b2, me.b2, other.b3, me.b3]
    const uint32_t sel1 = (lane & 1) ? 0x3726u : 0x5140u;
    // bit 1 clear: first pixel of the pair: [me.h0, other.h0]; set: second pixel: [other.h1, me.h1]
    const uint32_t sel2 = (lane & 2) ? 0x3276u : 0x5410u;
#pragma unroll
    for (int j = 0; j < WORDS; j++) {
        const uint32_t o1 = __shfl_xor_sync(0xffffffffu, w[j], 1);
        const uint32_t t = __byte_perm(w[j], o1, sel1);
        const uint32_t o2 = __shfl_xor_sync(0xffffffffu, t, 2);
        w[j] = __byte_perm(t, o2, sel2);
    }
}

// tmW: the weights / caller's B as an [N][K] K-contiguous matrix, box {cb, 128}.
// tmX: the activations / caller's A: tiled [M][K] map with box {128, b_rows} (CONV = false) or an im2col map over
//      NHWC activations with cb channels x b_rows pixels per load (CONV = true).
template <bool CONV, bool TWO_SM>
__global__ void __launch_bounds__(32 * (CONV ? 3 : 2) + 32 * SWAP_EPI_WARPS, 1)
gemm_i8_swap_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const SwapParams p) {
    constexpr int NPROD = CONV ? 2 : 1;
    constexpr int EPI_THREADS = 32 * SWAP_EPI_WARPS;
    constexpr int NTHREADS = 32 * (1 + NPROD) + EPI_THREADS;
    constexpr int PROD2_WARP = 2 + SWAP_EPI_WARPS;
    constexpr int TILE_CH = TWO_SM ? 2 * BM : BM;         // output channels per tile
    constexpr int A_BYTES = BM * BK;                      // weights per ring slot and CTA: 128 channels x 128 bytes of K

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sbase = raw + pad;
    const uint32_t sA = sbase, sB = sbase + p.off_b;
    const uint32_t bar_full = sbase + p.off_bar;
    const uint32_t bar_empty = bar_full + SWAP_MAX_STAGES * 8;
    const uint32_t bar_acc_full = bar_empty + SWAP_MAX_STAGES * 8;
    const uint32_t bar_acc_empty = bar_acc_full + 2 * 8;
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + p.off_bar + (2 * SWAP_MAX_STAGES + 4) * 8);
    volatile int* s_stop = reinterpret_cast<volatile int*>(smem + p.off_bar + (2 * SWAP_MAX_STAGES + 4) * 8 + 4);

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    const WaitEnv env{s_stop, p.dev_status, p.wait_limit_cycles};
    const uint32_t rank = TWO_SM ? cluster_ctarank() : 0u;
    const int stages = p.stages;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, TWO_SM ? 2 * SWAP_EPI_WARPS : EPI_THREADS);
        }
        *s_stop = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        if (TWO_SM) {
            tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(s_tmem)), (uint32_t)p.tmem_cols);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(const_cast<uint32_t*>(s_tmem)), (uint32_t)p.tmem_cols);
            tmem_relinquish();
        }
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmX);
    }
    // The next kernel of the stream may be scheduled from here on; this one goes on with set-up that touches only shared
    // and tensor memory, and waits for its own predecessor right before the roles start (below).
    grid_launch_dependents();
    uint32_t tmem_base = 0;
    if (TWO_SM) {
        tc_fence_before();
        cluster_sync_all();              // both CTAs' barriers exist before anything remote touches them
        tc_fence_after();
        tmem_base = __shfl_sync(0xffffffffu, *s_tmem, 0);
    } else if (warp == 0) {
        __syncwarp();
        named_barrier_arrive(15, NTHREADS);
    } else if (NPROD == 2 && warp == PROD2_WARP) {
        named_barrier(15, NTHREADS);
    } else {
        tc_fence_before();
        named_barrier(15, NTHREADS);
        tc_fence_after();
        tmem_base = __shfl_sync(0xffffffffu, *s_tmem, 0);
    }

    const KLoop kl = p.kl;
    const uint32_t a_sub_bytes = BM * kl.cb, b_sub_bytes = (uint32_t)p.b_rows * kl.cb;
    const int first_tile = TWO_SM ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int tile_step = TWO_SM ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const uint32_t full0 = TWO_SM ? map_to_cta(bar_full, 0) : bar_full;
    const uint32_t acc_empty0 = TWO_SM ? map_to_cta(bar_acc_empty, 0) : bar_acc_empty;
    const uint32_t tx_mult = TWO_SM ? 2u : 1u;
    // Global memory is read and written from here on: everything the preceding kernel wrote must be visible.
    grid_dependency_wait();

    if (warp == 0 || (NPROD == 2 && warp == PROD2_WARP)) {
        // ------------------------------------------------------------------ producer (whole warp loops, one lane issues)
        const int pid = warp == 0 ? 0 : 1;
        int stage = 0;
        uint32_t phase = 0, issued = 0, issued_phase = 0, seq = 0;     // seq: ring slots filled so far by both producers together
        bool ok = true, first_pass = true;
        const bool leader = elect_one();
        const uint32_t stage_tx = a_sub_bytes + b_sub_bytes;
        for (int tile = first_tile; ok && tile < p.num_tiles; tile += tile_step) {
            const int m_tile = fast_div(tile, p.n_blocks, p.inv_nb), n_blk = tile - m_tile * p.n_blocks;
            const int row_w = n_blk * TILE_CH + (int)rank * BM;              // this CTA's first channel
            const int row_x = m_tile * p.pw + (int)rank * p.b_rows;          // this CTA's first output row / pixel
            int w0 = 0, h0 = 0, img = 0;
            if (CONV) {
                const int pq = kl.P * kl.Q;
                img = fast_div(row_x, pq, kl.inv_pq);
                const int rem = row_x - img * pq;
                const int op = fast_div(rem, kl.Q, kl.inv_q), oq = rem - op * kl.Q;
                h0 = op * kl.stride_h - kl.pad_h;
                w0 = oq * kl.stride_w - kl.pad_w;
            }
            int c_idx = 0, fs = 0, fr = 0;
            for (int kbi = 0; kbi < kl.num_kblocks;) {
                const int nb = min(kl.nsub, kl.num_kblocks - kbi);
                if (NPROD == 2 && (seq & 1) != (uint32_t)pid) {
                    // the other producer's turn (turns alternate along the sequence of slots, so the ring may have an odd
                    // number of them): only keep the counters in step
                    for (int j = 0; j < nb; j++, kbi++)
                        if (CONV && ++c_idx == kl.cblocks) { c_idx = 0; if (++fs == kl.S) { fs = 0; ++fr; } }
                    ++seq;
                    if (++stage == stages) { stage = 0; phase ^= 1; first_pass = false; }
                    continue;
                }
                if (!first_pass && !mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1, env, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                const uint32_t full = full0 + 8 * stage;
                if (leader && rank == 0) mbar_expect_tx(bar_full + 8 * stage, tx_mult * nb * stage_tx);
                for (int j = 0; j < nb; j++, kbi++) {
                    const uint32_t dstA = sA + stage * A_BYTES + j * a_sub_bytes;
                    const uint32_t dstB = sB + stage * p.b_stage_bytes + j * b_sub_bytes;
                    if (leader) {
                        if (TWO_SM) tma_load_2d_pair(dstA, &tmW, full, kbi * kl.cb, row_w);
                        else tma_load_2d(dstA, &tmW, full, kbi * kl.cb, row_w);
                    }
                    if (CONV) {
                        if (leader) {
                            if (TWO_SM) tma_load_im2col_4d_pair(dstB, &tmX, full, c_idx * kl.cb, w0, h0, img, (uint16_t)fs, (uint16_t)fr);
                            else tma_load_im2col_4d(dstB, &tmX, full, c_idx * kl.cb, w0, h0, img, (uint16_t)fs, (uint16_t)fr);
                        }
                        if (++c_idx == kl.cblocks) { c_idx = 0; if (++fs == kl.S) { fs = 0; ++fr; } }
                    } else if (leader) {
                        if (TWO_SM) tma_load_2d_pair(dstB, &tmX, full, kbi * BK, row_x);
                        else tma_load_2d(dstB, &tmX, full, kbi * BK, row_x);
                    }
                }
                issued |= 1u << stage;
                issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
                ++seq;
                if (++stage == stages) { stage = 0; phase ^= 1; first_pass = false; }
            }
        }
        if (*s_stop && rank == 0) {
            // stopping early: let every copy this warp started land before the CTA retires
            for (int s = 0; s < stages; s++)
                if (issued & (1u << s))
                    if (!mbar_wait_drain(bar_full + 8 * s, (issued_phase >> s) & 1u, p.wait_limit_cycles))
                        atomicCAS(p.dev_status, 0u, (unsigned)DEV_TIMEOUT_DRAIN);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (whole warp loops, one lane issues)
        const uint32_t idesc = make_idesc_i8(TILE_CH, p.pw, 0, 0);
        const uint64_t swz = kl.cb == 128 ? SWZ_128B : (kl.cb == 64 ? SWZ_64B : SWZ_32B);
        const uint64_t desc_hi = make_smem_desc(0, 16, 8 * kl.cb, swz);
        const bool leader = elect_one();
        const int per_sub = kl.cb / UMMA_K;
        uint32_t offA[4], offB[4];
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const int sub = i / per_sub, k = i - sub * per_sub;
            offA[i] = (sub * a_sub_bytes + k * UMMA_K) >> 4;
            offB[i] = (sub * b_sub_bytes + k * UMMA_K) >> 4;
        }
        const uint32_t a_base = (sA & 0x3FFFFu) >> 4, b_base = (sB & 0x3FFFFu) >> 4;
        int stage = 0, ab = 0;
        uint32_t phase = 0, acc_phase = 0;
        bool ready = false, ok = rank == 0;              // in a pair only the even CTA issues
        for (int tile = first_tile; ok && tile < p.num_tiles; tile += tile_step) {
            if (!mbar_wait_warp(bar_acc_empty + 8 * ab, acc_phase ^ 1, env, DEV_TIMEOUT_MMA_ACC)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + ab * p.pw;
            for (int it = 0; it < kl.num_iters; it++) {
                if (!ready && !mbar_wait_warp(bar_full + 8 * stage, phase, env, DEV_TIMEOUT_MMA_FULL)) { ok = false; break; }
                tc_fence_after();
                int nstage = stage + 1;
                uint32_t nphase = phase;
                if (nstage == stages) { nstage = 0; nphase ^= 1; }
                const bool peek = mbar_test_wait(bar_full + 8 * nstage, nphase);
                if (leader) {
                    const int nm = it == kl.num_iters - 1 ? kl.mmas_last : 4;
                    const uint32_t a0 = a_base + stage * (A_BYTES >> 4);
                    const uint32_t b0 = b_base + stage * ((uint32_t)p.b_stage_bytes >> 4);
#pragma unroll
                    for (int i = 0; i < 4; i++)
                        if (i < nm) {
                            if (TWO_SM) mma_i8_ss_pair(d_tmem, desc_hi | (uint64_t)(a0 + offA[i]), desc_hi | (uint64_t)(b0 + offB[i]), idesc,
                                                       (it | i) != 0 ? 1u : 0u);
                            else mma_i8_ss(d_tmem, desc_hi | (uint64_t)(a0 + offA[i]), desc_hi | (uint64_t)(b0 + offB[i]), idesc,
                                           (it | i) != 0 ? 1u : 0u);
                        }
                    if (TWO_SM) tc_commit_pair(bar_empty + 8 * stage);
                    else tc_commit(bar_empty + 8 * stage);
                }
                ready = __all_sync(0xffffffffu, peek);
                stage = nstage;
                phase = nphase;
            }
            if (!ok) break;
            if (leader) {
                if (TWO_SM) tc_commit_pair(bar_acc_full + 8 * ab);
                else tc_commit(bar_acc_full + 8 * ab);
            }
            ab ^= 1;
            if (ab == 0) acc_phase ^= 1;
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue: one output channel per thread
        const int quarter = warp & 3;                   // a warp may only read lanes 32*(warp%4) .. +31
        const int cgroup = (warp - 2) >> 2;             // which share of the strip's columns this warp handles
        constexpr int GROUPS = SWAP_EPI_WARPS / 4;
        const int units = p.pw / SWAP_UNIT;             // 16-pixel column units, dealt to the groups as evenly as they go
        const int u_base = units / GROUPS, u_rem = units % GROUPS;
        const int col_begin = SWAP_UNIT * (cgroup * u_base + min(cgroup, u_rem));
        const int col_end = col_begin + SWAP_UNIT * (u_base + (cgroup < u_rem ? 1 : 0));
        const int pix = swap_pixel_of_lane(lane);       // after the transpose: which pixel of each group of four this lane holds
        const int64_t row4 = 4 * p.ldc;                 // four rows of C
        int ab = 0, cached_n_blk = -1;
        uint32_t acc_phase = 0;
        bool dead = false;
        SwapChan ch = make_swap_chan(0, 0, 0, 0);
        bool all_fold = false;
        int n = 0;
        for (int tile = first_tile; tile < p.num_tiles; tile += tile_step) {
            const int m_tile = fast_div(tile, p.n_blocks, p.inv_nb), n_blk = tile - m_tile * p.n_blocks;
            if (n_blk != cached_n_blk) {
                // this thread's channel changed: three loads, before the wait so that they overlap the main loop
                n = n_blk * TILE_CH + (int)rank * BM + quarter * 32 + lane;
                int32_t bias = 0, mult = 0, shift = 0;
                float fs = 0.f;
                if (n < p.N) {
                    bias = p.bias ? p.bias[n] : 0;
                    if (p.fscale) fs = p.fscale[p.per_channel ? n : 0];
                    else { mult = p.mult[p.per_channel ? n : 0]; shift = p.shift[p.per_channel ? n : 0]; }
                }
                ch = make_swap_chan(bias, mult, shift, p.relu);
                if (p.fscale) { ch.form = 3; ch.fscale = fs; }
                all_fold = __all_sync(0xffffffffu, ch.form == 0);
                cached_n_blk = n_blk;
            }
            if (!dead) dead = !__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * ab, acc_phase, env, DEV_TIMEOUT_EPILOGUE));
            if (dead) continue;
            tc_fence_after();
            const int m0 = m_tile * p.pw;
            const int n_warp = n_blk * TILE_CH + (int)rank * BM + quarter * 32;       // first channel of this warp
            const int n_quad = n_warp + (lane & ~3);                                    // first channel of this lane's quad
            const uint32_t t0 = tmem_base + ab * p.pw + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
            for (int col = col_begin; col < col_end; col += 32) {
                const int width = min(32, col_end - col);                  // 32, or 16 in a group's last chunk
                if (m0 + col >= p.M || n_warp >= p.N) break;               // nothing of this chunk (or warp) is inside C
                int32_t v[32];
                uint32_t out[8];
                if (width == 32) {
                    tmem_ld_32x32(t0 + col, v);
                    tmem_ld_wait();
                    swap_requant<32>(v, ch, p.relu, all_fold, out);
                } else {
                    tmem_ld_32x16(t0 + col, v);
                    tmem_ld_wait();
                    swap_requant<16>(v, ch, p.relu, all_fold, out);
                }
                if (p.c_word_ok) {
                    // word j: channels n_quad .. n_quad + 3 of output row m0 + col + 4j + pix
                    if (width == 32) quad_transpose<8>(out, lane);
                    else quad_transpose<4>(out, lane);
                    if (n_quad < p.N) {                                    // N is a multiple of 4: a quad is inside or outside as a whole
                        int8_t* cp = p.C + (int64_t)(m0 + col + pix) * p.ldc + n_quad;
                        const int rows_left = p.M - (m0 + col + pix);      // rows of C from this lane's first row to the end
#pragma unroll
                        for (int j = 0; j < 8; j++) {
                            if (4 * j < width && 4 * j < rows_left) *reinterpret_cast<uint32_t*>(cp) = out[j];
                            cp += row4;
                        }
                    }
                } else if (n < p.N) {
                    int8_t* cp = p.C + (int64_t)(m0 + col) * p.ldc + n;
#pragma unroll
                    for (int j = 0; j < 32; j++)
                        if (j < width && m0 + col + j < p.M) cp[(int64_t)j * p.ldc] = (int8_t)(out[j >> 2] >> (8 * (j & 3)));
                }
            }
            tc_fence_before();
            if (TWO_SM) {
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(acc_empty0 + 8 * ab);
            } else {
                mbar_arrive(bar_acc_empty + 8 * ab);
            }
            ab ^= 1;
            if (ab == 0) acc_phase ^= 1;
        }
    }

    tc_fence_before();
    if (TWO_SM) {
        cluster_sync_all();
        if (warp == 1) {
            tc_fence_after();
            tmem_dealloc_pair(tmem_base, (uint32_t)p.tmem_cols);
        }
    } else {
        __syncthreads();
        if (warp == 1) {
            tc_fence_after();
            tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
        }
    }
}

}  // namespace i8
