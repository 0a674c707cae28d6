// Stride-1 convolution with the input slab kept in shared memory ("load once, reuse across filter taps").
//
// The implicit-GEMM path fetches every input pixel once per filter tap (R*S times) through im2col TMA loads; for
// layers with few filters that traffic from L2 bounds the kernel.  Here a tile is TH whole output rows of one image,
// laid out as a raster of width Wp = W + 2*pad_w (the padded input width), and ONE tiled TMA load per channel block
// brings the (TH + R - 1) x Wp input pixels the tile needs into shared memory, zero padding included (out-of-bounds
// fill).  In that raster the input pixel of output position j under filter tap (r, s) is simply row j + r*Wp + s, so
// the A operand of tap (r, s) is the same slab read through a descriptor whose start address is moved by (r*Wp + s)
// rows: the tensor core applies the swizzle to absolute shared-memory address bits, exactly as the TMA engine did
// when it wrote the rows, so any whole-row offset is legal (measured: every row offset reads back the right bytes for
// the 32-, 64- and 128-byte swizzles with a zero base-offset field).  Output positions in the Wp - Q padding columns
// are computed and dropped.  The filter bank stays resident in shared memory for the whole kernel (the paper's "load
// B once" step, Code Examples appendix).
//
// This is the paper's data-movement theme (Evaluation, "minimizing data movement between main memory and the
// accelerator-local memories") applied to the B200 memory hierarchy.  Roles, barriers and bounded waits are those of
// gemm_tc.cuh, except that two warps issue MMAs (one per accumulator).
#pragma once
#include "gemm_tc.cuh"

namespace i8 {

constexpr int SLAB_MAX_STAGES = 8;
constexpr int SLAB_THREADS = 32 * 3 + 32 * 8;     // producer, MMA issuer, 8 epilogue warps, second MMA issuer
constexpr int SLAB_ISSUER2_WARP = 10;
constexpr int SLAB_ACC = 4;                       // accumulators: the issuers may run this many tiles ahead of the read-out

struct ConvSlabParams {
    int8_t* y;
    const int32_t* bias;
    const int32_t* mult;
    const int32_t* shift;
    int per_channel, relu;
    int Kf;                          // filters = output channels (<= BN)
    int P, Q;                        // output extent per image
    int R, S;
    int Wp;                          // raster width: W + 2 * pad_w
    int TH;                          // output rows per tile: floor(128 / Wp)
    int pad_h, pad_w;
    int cb, cblocks;                 // channel block in bytes (128, 64 or 32) and C / cb
    int tiles_per_img, num_tiles;    // ceil(P / TH), images * tiles_per_img
    uint32_t inv_tpi, inv_wp;        // floor(2^32 / tiles_per_img), floor(2^32 / Wp) (0xffffffff for a divisor of 1)
    int slab_tx_bytes;               // bytes one slab load delivers: cb * Wp * (TH + R - 1)
    int stage_bytes;                 // distance between ring slots (multiple of 1024, covers the furthest row a tap reads)
    int stages;                      // ring slots (2 .. SLAB_MAX_STAGES)
    int off_b, off_const, off_bar;   // shared-memory offsets from the 1024-byte aligned base
    int y_vec_ok;                    // y and Kf are 16-byte aligned: full chunks go out as 16-byte stores
    long long wait_limit_cycles;
    unsigned* dev_status;
};

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* m, uint32_t bar, int c, int w, int h, int n) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(c), "r"(w), "r"(h), "r"(n)
        : "memory");
}

// tmX: tiled map over the NHWC activations, dims {C, W, H, N}, box {cb, Wp, TH + R - 1, 1}.
// tmW: the filter bank as a [Kf][R*S*C] matrix, box {cb, BN}.
// TAPS = R*S when the filter size is known at compile time (9: the tap offsets and filter descriptors then live in
// registers and the issue loop is fully unrolled), 0 for any other filter.
template <int BN, int TAPS>
__global__ void __launch_bounds__(SLAB_THREADS, 1)
conv_slab_i8_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const ConvSlabParams p) {
    constexpr int EPI_THREADS = 256;
    static_assert(BN == 64 || BN == 128, "filter tiles of 64 or 128");
    constexpr int TMEM_COLS = SLAB_ACC * BN;         // 256 or 512 columns

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sbase = raw + pad;
    const uint32_t sSlab = sbase, sB = sbase + p.off_b;
    int32_t* s_m2 = reinterpret_cast<int32_t*>(smem + p.off_const);
    int32_t* s_bias = s_m2 + BN;
    int32_t* s_lo = s_bias + BN;
    int32_t* s_hi = s_lo + BN;
    int32_t* s_mult = s_hi + BN;
    int32_t* s_shift = s_mult + BN;
    int32_t* s_rnd = s_shift + BN;
    long long* s_c64 = reinterpret_cast<long long*>(s_rnd + BN);
    const uint32_t bar_full = sbase + p.off_bar;
    const uint32_t bar_empty = bar_full + SLAB_MAX_STAGES * 8;
    const uint32_t bar_acc_full = bar_empty + SLAB_MAX_STAGES * 8;
    const uint32_t bar_acc_empty = bar_acc_full + SLAB_ACC * 8;
    const uint32_t bar_w = bar_acc_empty + SLAB_ACC * 8;
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + p.off_bar + (2 * SLAB_MAX_STAGES + 2 * SLAB_ACC + 1) * 8);
    volatile int* s_stop = reinterpret_cast<volatile int*>(smem + p.off_bar + (2 * SLAB_MAX_STAGES + 2 * SLAB_ACC + 1) * 8 + 4);

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    const WaitEnv env{s_stop, p.dev_status, p.wait_limit_cycles};
    const int stages = p.stages;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < SLAB_ACC; b++) {
            mbar_init(bar_acc_full + 8 * b, 1);
            mbar_init(bar_acc_empty + 8 * b, EPI_THREADS / 2);     // the four warps of the group that reads the tile out
        }
        mbar_init(bar_w, 1);
        *s_stop = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(s_tmem)), TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmX);
        tma_prefetch_desc(&tmW);
    }
    grid_launch_dependents();        // the next kernel may be scheduled; this one waits for its predecessor after set-up
    // Set-up barrier.  The producer warp initialised the mbarriers itself and needs nothing from the others, so it only
    // signals and starts loading at once; everybody else waits for the barriers and the tensor-memory address.
    uint32_t tmem_base = 0;
    if (warp == 0) {
        __syncwarp();
        named_barrier_arrive(15, SLAB_THREADS);
    } else {
        tc_fence_before();
        named_barrier(15, SLAB_THREADS);
        tc_fence_after();
        tmem_base = __shfl_sync(0xffffffffu, *s_tmem, 0);
    }

    const int taps = p.R * p.S;
    const uint32_t w_sub_bytes = BN * p.cb;          // one (tap, channel block) of the filter bank
    grid_dependency_wait();          // global memory is touched from here on

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        const bool leader = elect_one();
        int stage = 0;
        uint32_t phase = 0, issued = 0, issued_phase = 0;
        bool ok = true, w_issued = false;
        for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x) {
            const int img = fast_div(tile, p.tiles_per_img, p.inv_tpi);
            const int p0 = (tile - img * p.tiles_per_img) * p.TH;
            for (int c = 0; c < p.cblocks; c++) {
                if (!mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1, env, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                if (leader) {
                    mbar_expect_tx(bar_full + 8 * stage, (uint32_t)p.slab_tx_bytes);
                    // rows p0 - pad_h .. and columns -pad_w .. : everything outside the image arrives as zeros
                    tma_load_4d(sSlab + stage * p.stage_bytes, &tmX, bar_full + 8 * stage, c * p.cb, -p.pad_w, p0 - p.pad_h, img);
                }
                issued |= 1u << stage;
                issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
                if (++stage == stages) { stage = 0; phase ^= 1; }
            }
            if (ok && tile == (int)blockIdx.x && leader) {
                // the whole filter bank, once, right behind the first tile's slabs: sub-tile (tap t, channel block c)
                // holds w[:, t, c*cb .. c*cb + cb)
                mbar_expect_tx(bar_w, (uint32_t)(taps * p.cblocks) * w_sub_bytes);
                for (int t = 0; t < taps; t++)
                    for (int c = 0; c < p.cblocks; c++)
                        tma_load_2d(sB + (t * p.cblocks + c) * w_sub_bytes, &tmW, bar_w, (t * p.cblocks + c) * p.cb, 0);
                w_issued = true;
            }
        }
        w_issued = __any_sync(0xffffffffu, w_issued);
        if (*s_stop) {
            // stopping early: let every copy this warp started land before the CTA retires
            if (w_issued && !mbar_wait_drain(bar_w, 0, p.wait_limit_cycles)) atomicCAS(p.dev_status, 0u, (unsigned)DEV_TIMEOUT_DRAIN);
            for (int s = 0; s < stages; s++)
                if (issued & (1u << s))
                    if (!mbar_wait_drain(bar_full + 8 * s, (issued_phase >> s) & 1u, p.wait_limit_cycles))
                        atomicCAS(p.dev_status, 0u, (unsigned)DEV_TIMEOUT_DRAIN);
        }
        __syncwarp();
    } else if (warp == 1 || warp == SLAB_ISSUER2_WARP) {
        // ------------------------------------------------------------------ MMA issuers
        // Two warps issue: warp 1 the even tiles of this CTA's sequence (even accumulators), the last warp the odd ones
        // (odd accumulators).  A 128 x 64 x 32 instruction lasts ~50 cycles and the tensor core's queue is short, so
        // one thread's barrier round trips between tiles would leave the tensor core idle; two independent streams
        // into different accumulators fill each other's gaps.
        const int iss = warp == 1 ? 0 : 1;
        constexpr uint32_t idesc = make_idesc_i8(BM, BN, 0, 0);
        const uint64_t swz = p.cb == 128 ? SWZ_128B : (p.cb == 64 ? SWZ_64B : SWZ_32B);
        const uint64_t desc_hi = make_smem_desc(0, 16, 8 * p.cb, swz);       // rows cb bytes apart, 8-row groups 8*cb apart
        const bool leader = elect_one();
        const int ksteps = p.cb / UMMA_K;
        // Descriptor arithmetic happens on the low word only (the start-address field, in 16-byte units; the offsets
        // below never carry out of it).
        const uint32_t desc_hi32 = (uint32_t)(desc_hi >> 32), desc_lo32 = (uint32_t)desc_hi;
        const uint64_t hi = (uint64_t)desc_hi32 << 32;
        const uint32_t row_units = (uint32_t)p.cb >> 4;                     // one raster row
        const uint32_t row_skip = (uint32_t)(p.Wp - p.S) * row_units;       // from the end of one filter row to the next
        const uint32_t tap_units = (uint32_t)p.cblocks * (w_sub_bytes >> 4);// from one tap's filter sub-tile to the next
        const uint32_t b_base = desc_lo32 + ((sB & 0x3FFFFu) >> 4);
        // known filter size: per tap, the slab row offset and the filter sub-tile's descriptor word, kept in registers
        uint32_t tap_a[TAPS > 0 ? TAPS : 1], tap_b[TAPS > 0 ? TAPS : 1];
        if (TAPS > 0) {
#pragma unroll
            for (int t = 0; t < (TAPS > 0 ? TAPS : 1); t++) {
                const int r = t / p.S, s = t - r * p.S;
                tap_a[t] = (uint32_t)(r * p.Wp + s) * row_units;
                tap_b[t] = b_base + (uint32_t)t * tap_units;
            }
        }
        int ab = iss;
        const int first = (int)blockIdx.x + iss * (int)gridDim.x;        // this issuer's first tile; it takes every second one
        int stage = 0;
        uint32_t phase = 0, acc_phase = 0;
        for (int c = 0; c < iss * p.cblocks; c++)                        // skip the ring slots of the other issuer's first tile
            if (++stage == stages) { stage = 0; phase ^= 1; }
        bool ok = first >= p.num_tiles || mbar_wait_warp(bar_w, 0, env, DEV_TIMEOUT_MMA_FULL);
        for (int tile = first; ok && tile < p.num_tiles; tile += 2 * (int)gridDim.x) {
            if (!mbar_wait_warp(bar_acc_empty + 8 * ab, acc_phase ^ 1, env, DEV_TIMEOUT_MMA_ACC)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + ab * BN;
            for (int c = 0; c < p.cblocks; c++) {
                if (!mbar_wait_warp(bar_full + 8 * stage, phase, env, DEV_TIMEOUT_MMA_FULL)) { ok = false; break; }
                tc_fence_after();
                if (leader && TAPS > 0) {
                    const uint32_t a_lo = desc_lo32 + (((sSlab + stage * p.stage_bytes) & 0x3FFFFu) >> 4);
                    const uint32_t b_lo = (uint32_t)c * (w_sub_bytes >> 4);
#pragma unroll
                    for (int t = 0; t < (TAPS > 0 ? TAPS : 1); t++) {
#pragma unroll
                        for (int k = 0; k < 4; k++)
                            if (k < ksteps) {
                                // the tile's very first instruction overwrites the accumulator
                                if (t == 0 && k == 0) mma_i8_ss(d_tmem, hi | (a_lo + tap_a[0]), hi | (b_lo + tap_b[0]), idesc, c == 0 ? 0u : 1u);
                                else mma_i8_ss_acc(d_tmem, hi | (a_lo + tap_a[t] + 2 * k), hi | (b_lo + tap_b[t] + 2 * k), idesc);
                            }
                    }
                    tc_commit(bar_empty + 8 * stage);        // slab reusable once these instructions have read it
                } else if (leader) {
                    uint32_t a_lo = desc_lo32 + (((sSlab + stage * p.stage_bytes) & 0x3FFFFu) >> 4);
                    uint32_t b_lo = b_base + (uint32_t)c * (w_sub_bytes >> 4);
                    uint32_t accum = c == 0 ? 0u : 1u;
                    for (int r = 0; r < p.R; r++, a_lo += row_skip)
                        for (int s = 0; s < p.S; s++, a_lo += row_units, b_lo += tap_units) {
#pragma unroll
                            for (int k = 0; k < 4; k++)
                                if (k < ksteps) {
                                    mma_i8_ss(d_tmem, hi | (a_lo + 2 * k), hi | (b_lo + 2 * k), idesc, accum);
                                    accum = 1u;
                                }
                        }
                    tc_commit(bar_empty + 8 * stage);
                }
                __syncwarp();
                if (++stage == stages) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            if (leader) tc_commit(bar_acc_full + 8 * ab);
            __syncwarp();
            ab += 2;
            if (ab >= SLAB_ACC) { ab -= SLAB_ACC; acc_phase ^= 1; }
            for (int c = 0; c < p.cblocks; c++)                          // the other issuer's tile in between
                if (++stage == stages) { stage = 0; phase ^= 1; }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue
        const int etid = threadIdx.x - 64;
        const int quarter = warp & 3;                   // a warp may only read lanes 32*(warp%4) .. +31
        // The two groups of four warps take alternate tiles (all BN columns each), so that one tile's tensor-memory load
        // and stores overlap the other's arithmetic: a warp's chunk is one dependent chain, and with both groups on the same
        // tile the read-outs ran one after the other at 0.8-1.0 us per tile while the issuers were 1.5 us ahead
        // (measured: 10.05 -> 9.15 us on the 56x56x64 -> 64 layer; four groups on 16 warps: 9.0 us, not kept).
        const int tgroup = (warp - 2) >> 2;
        // per-channel constants of the (single) block of filters, prepared while the first slab is in flight
        bool all32 = true, allfold = true;
        for (int c = etid; c < BN; c += EPI_THREADS) {
            int32_t bias = 0, mult = 0, shift = 0;
            if (c < p.Kf) {
                bias = p.bias ? p.bias[c] : 0;
                mult = p.mult[p.per_channel ? c : 0];
                shift = p.shift[p.per_channel ? c : 0];
            }
            const ChanConst cc = make_chan_const(mult, shift, p.relu);
            s_bias[c] = bias; s_lo[c] = cc.lo; s_hi[c] = cc.hi;
            s_mult[c] = cc.mult; s_shift[c] = cc.shift; s_rnd[c] = cc.rnd;
            int32_t m2;
            const bool ok32 = make_shift32_mult(mult, shift, m2);
            all32 = ok32 && all32;
            allfold = allfold && ok32 && (!p.relu || m2 >= 0);
            s_m2[c] = m2;
            s_c64[c] = make_fold_addend(bias, m2);
        }
        const bool shift32 = named_barrier_and(2, EPI_THREADS, all32);
        const bool fold = named_barrier_and(3, EPI_THREADS, allfold);
        // position of this thread's accumulator row in the tile's raster: (dy, dx) = (j / Wp, j % Wp)
        const int j = quarter * 32 + lane;
        const int dy = fast_div(j, p.Wp, p.inv_wp), dx = j - dy * p.Wp;
        const bool in_raster = dy < p.TH && dx < p.Q;
        int ab = 0, seq = 0;
        uint32_t acc_phase = 0;
        bool dead = false;
        for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x, seq++) {
            if ((seq & 1) != tgroup) {                    // the other group's tile
                if (++ab == SLAB_ACC) { ab = 0; acc_phase ^= 1; }
                continue;
            }
            const int img = fast_div(tile, p.tiles_per_img, p.inv_tpi);
            const int p0 = (tile - img * p.tiles_per_img) * p.TH;
            // A warp whose wait expired stays in the loop without touching the accumulators; the stop flag it raised
            // ends the other roles.
            if (!dead) dead = !__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * ab, acc_phase, env, DEV_TIMEOUT_EPILOGUE));
            if (dead) continue;
            tc_fence_after();
            const bool live = in_raster && p0 + dy < p.P;
            int8_t* yrow = p.y + ((int64_t)(img * p.P + p0 + dy) * p.Q + dx) * p.Kf;
            const uint32_t t0 = tmem_base + ab * BN + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
            for (int ch = 0; ch < BN / 32; ch++) {
                const int c0 = ch * 32;
                if (c0 >= p.Kf) break;
                int32_t v[32];
                tmem_ld_32x32(t0 + c0, v);
                tmem_ld_wait();
                uint32_t out[8];
                if (fold) {
                    if (p.relu) epilogue_chunk_fold_add<true>(v, s_bias, s_m2, c0, out);
                    else epilogue_chunk_fold_add<false>(v, s_bias, s_m2, c0, out);
                } else if (shift32) {
                    if (p.relu) epilogue_chunk_shift32<true>(v, s_bias, s_m2, c0, out);
                    else epilogue_chunk_shift32<false>(v, s_bias, s_m2, c0, out);
                } else {
                    epilogue_chunk(v, s_bias, s_lo, s_hi, s_mult, s_shift, s_rnd, c0, out);
                }
                if (live) store_row_chunk(yrow, c0, p.Kf, p.y_vec_ok != 0, out);
            }
            tc_fence_before();
            mbar_arrive(bar_acc_empty + 8 * ab);
            if (++ab == SLAB_ACC) { ab = 0; acc_phase ^= 1; }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace i8
