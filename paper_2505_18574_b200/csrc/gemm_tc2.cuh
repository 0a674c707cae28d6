// Two-SM variant of the large-tile GEMM: a cluster of two CTAs computes one 256 x 256 output tile with
// tcgen05.mma.cta_group::2 (256 x 256 x 32 per instruction, issued by one thread of the even CTA).
//
// Each CTA holds 128 rows of A and 128 of the tile's 256 B rows (columns of the output); the hardware feeds
// both SMs' tensor cores from both shared memories, and each SM accumulates its own 128 x 256 half of the
// tile in its own tensor memory.  Per 128 bytes of K a CTA therefore fetches 32 KiB instead of the 48 KiB of
// the one-SM kernel (two thirds of the L2 and shared-memory traffic for the same products), and one issuing
// thread drives two tensor cores.
//
//   warp 0      producer : both CTAs; TMA loads (cta_group::2 form) complete on the EVEN CTA's "full" barrier
//   warp 1      MMA      : even CTA only; commits are multicast to the barriers of both CTAs
//   warps 2..9  epilogue : both CTAs read their own accumulator half; one lane per warp then arrives on the
//                          even CTA's "accumulator free" barrier (remotely from the odd CTA)
//
// No load uses cluster multicast.  Every wait is bounded as in the one-SM kernel; the two CTAs meet at a
// cluster barrier after set-up and before tensor memory is released.
#pragma once
#include "gemm_tc.cuh"

namespace i8 {

constexpr int TC2_STAGES = 6;
constexpr int TC2_BN = 256;
constexpr int TC2_EPI_WARPS = 8;
constexpr int TC2_THREADS = 64 + 32 * TC2_EPI_WARPS;

struct Tc2Smem {
    static constexpr int A_BYTES = BM * BK;                 // this CTA's 128 rows of A
    static constexpr int B_BYTES = (TC2_BN / 2) * BK;       // this CTA's half of the B tile
    static constexpr int OFF_A = 0;
    static constexpr int OFF_B = OFF_A + TC2_STAGES * A_BYTES;
    static constexpr int OFF_CONST = OFF_B + TC2_STAGES * B_BYTES;
    static constexpr int OFF_BAR = OFF_CONST + 7 * TC2_BN * 4;   // full[S], empty[S], acc_full[2], acc_empty[2]
    static constexpr int OFF_MISC = OFF_BAR + (2 * TC2_STAGES + 4) * 8;
    static constexpr int TOTAL = OFF_MISC + 16;
    static constexpr int DYN_BYTES = TOTAL + 1024;
    static constexpr int TMEM_COLS = 2 * TC2_BN;
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {   // every thread of both CTAs
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion may be counted on a barrier of either CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* m, uint32_t bar_cluster_addr, int x, int y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar_cluster_addr), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void mma_i8_ss_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on the barrier at the same shared-memory offset in both CTAs once the MMAs issued so far have finished.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC2_THREADS, 1)
gemm_i8_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmTcParams p) {
    using L = Tc2Smem;
    constexpr int STAGES = TC2_STAGES, BN = TC2_BN, EPI_WARPS = TC2_EPI_WARPS;
    constexpr int COLS_PER_GROUP = BN / (EPI_WARPS / 4);
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sbase = raw + pad;
    const uint32_t sA = sbase + L::OFF_A, sB = sbase + L::OFF_B;
    int32_t* s_m2 = reinterpret_cast<int32_t*>(smem + L::OFF_CONST);
    int32_t* s_bias = s_m2 + BN;
    int32_t* s_lo = s_bias + BN;
    int32_t* s_hi = s_lo + BN;
    int32_t* s_mult = s_hi + BN;
    int32_t* s_shift = s_mult + BN;
    int32_t* s_rnd = s_shift + BN;
    const uint32_t bar_full = sbase + L::OFF_BAR;
    const uint32_t bar_empty = bar_full + STAGES * 8;
    const uint32_t bar_acc_full = bar_empty + STAGES * 8;
    const uint32_t bar_acc_empty = bar_acc_full + 2 * 8;
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_MISC);
    volatile int* s_stop = reinterpret_cast<volatile int*>(smem + L::OFF_MISC + 4);

    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();           // 0 = even CTA (issues the MMAs), 1 = odd CTA
    const WaitEnv env{s_stop, p.dev_status, p.wait_limit_cycles};

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) {
            mbar_init(bar_full + 8 * s, 1);            // used in the even CTA: its producer's expect_tx arrival
            mbar_init(bar_empty + 8 * s, 1);           // in each CTA: one multicast commit
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(bar_acc_full + 8 * b, 1);        // in each CTA: one multicast commit
            mbar_init(bar_acc_empty + 8 * b, 2 * EPI_WARPS);   // used in the even CTA: one lane of every epilogue warp of both CTAs
        }
        *s_stop = 0;
        fence_barrier_init();
    }
    if (warp == 1) {                                   // the same warp in both CTAs, the same slot address
        tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(s_tmem)), L::TMEM_COLS);
        tmem_relinquish_pair();
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    tc_fence_before();
    cluster_sync_all();                                // both CTAs' barriers exist before anything remote touches them
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *s_tmem, 0);

    const TileSched sched = p.sched;                   // tiles of 256 x 256; this CTA owns rows rank*128 .. +127 of each
    const int num_kb = (p.K + BK - 1) / BK;
    const int mmas_last = ((p.K - (num_kb - 1) * BK) + UMMA_K - 1) / UMMA_K;
    const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer (both CTAs)
        int stage = 0;
        uint32_t phase = 0, issued = 0, issued_phase = 0;
        const bool leader = elect_one();
        const uint32_t full0 = map_to_cta(bar_full, 0);        // the even CTA's "full" barriers
        bool ok = true;
        for (int tile = cluster_id; ok && tile < sched.num_tiles; tile += num_clusters) {
            int m_blk, n_blk;
            sched.map(tile, m_blk, n_blk);
            const int row_a = m_blk * 256 + (int)rank * BM;
            const int row_b = n_blk * BN + (int)rank * (BN / 2);
            for (int kb = 0; kb < num_kb; kb++) {
                if (!mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1, env, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                if (leader) {
                    if (rank == 0) mbar_expect_tx(bar_full + 8 * stage, 2 * (L::A_BYTES + L::B_BYTES));   // both CTAs' bytes
                    tma_load_2d_pair(sA + stage * L::A_BYTES, &tmA, full0 + 8 * stage, kb * BK, row_a);
                    tma_load_2d_pair(sB + stage * L::B_BYTES, &tmB, full0 + 8 * stage, kb * BK, row_b);
                }
                issued |= 1u << stage;
                issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
        }
        if (*s_stop && rank == 0) {
            // stopping early: let the copies counted on this CTA's barriers land (they include the odd CTA's)
            for (int s = 0; s < STAGES; s++)
                if (issued & (1u << s))
                    if (!mbar_wait_drain(bar_full + 8 * s, (issued_phase >> s) & 1u, p.wait_limit_cycles))
                        atomicCAS(p.dev_status, 0u, (unsigned)DEV_TIMEOUT_DRAIN);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (even CTA only)
        if (rank == 0) {
            constexpr uint32_t idesc = make_idesc_i8(256, BN, 0, 0);
            const uint64_t desc_hi = make_smem_desc(0, 16, 1024, SWZ_128B);
            const bool leader = elect_one();
            const uint32_t a_base = (sA & 0x3FFFFu) >> 4, b_base = (sB & 0x3FFFFu) >> 4;
            int stage = 0, ab = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ready = false, ok = true;
            for (int tile = cluster_id; ok && tile < sched.num_tiles; tile += num_clusters) {
                if (!mbar_wait_warp(bar_acc_empty + 8 * ab, acc_phase ^ 1, env, DEV_TIMEOUT_MMA_ACC)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + ab * BN;
                for (int it = 0; it < num_kb; it++) {
                    if (!ready && !mbar_wait_warp(bar_full + 8 * stage, phase, env, DEV_TIMEOUT_MMA_FULL)) { ok = false; break; }
                    tc_fence_after();
                    int nstage = stage + 1;
                    uint32_t nphase = phase;
                    if (nstage == STAGES) { nstage = 0; nphase ^= 1; }
                    const bool peek = mbar_test_wait(bar_full + 8 * nstage, nphase);
                    if (leader) {
                        const int nm = it == num_kb - 1 ? mmas_last : 4;
                        const uint32_t a0 = a_base + stage * (L::A_BYTES >> 4), b0 = b_base + stage * (L::B_BYTES >> 4);
#pragma unroll
                        for (int i = 0; i < 4; i++)
                            if (i < nm)
                                mma_i8_ss_pair(d_tmem, desc_hi | (uint64_t)(a0 + 2 * i), desc_hi | (uint64_t)(b0 + 2 * i), idesc,
                                               (it | i) != 0 ? 1u : 0u);
                        tc_commit_pair(bar_empty + 8 * stage);     // frees the slot in both CTAs
                    }
                    ready = __all_sync(0xffffffffu, peek);
                    stage = nstage;
                    phase = nphase;
                }
                if (!ok) break;
                if (leader) tc_commit_pair(bar_acc_full + 8 * ab);  // both halves of the accumulator are complete
                ab ^= 1;
                if (ab == 0) acc_phase ^= 1;
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue (both CTAs, own accumulator half)
        const int etid = threadIdx.x - 64;
        const int quarter = warp & 3;
        const int cgroup = (warp - 2) >> 2;
        constexpr int EPI_THREADS = 32 * EPI_WARPS;
        const uint32_t acc_empty0 = map_to_cta(bar_acc_empty, 0);
        int ab = 0, cached_n_blk = -1;
        bool shift32 = false, dead = false;
        uint32_t acc_phase = 0;
        for (int tile = cluster_id; tile < sched.num_tiles; tile += num_clusters) {
            int m_blk, n_blk;
            sched.map(tile, m_blk, n_blk);
            const int n0 = n_blk * BN;
            if (n_blk != cached_n_blk) {
                named_barrier(1, EPI_THREADS);
                bool all32 = true;
                for (int c = etid; c < BN; c += EPI_THREADS) {
                    const int n = n0 + c;
                    int32_t bias = 0, mult = 0, shift = 0;
                    if (n < p.N && !p.raw) {
                        bias = p.bias ? p.bias[n] : 0;
                        mult = p.mult[p.per_channel ? n : 0];
                        shift = p.shift[p.per_channel ? n : 0];
                    }
                    const ChanConst cc = make_chan_const(mult, shift, p.relu);
                    s_bias[c] = bias; s_lo[c] = cc.lo; s_hi[c] = cc.hi;
                    s_mult[c] = cc.mult; s_shift[c] = cc.shift; s_rnd[c] = cc.rnd;
                    int32_t m2;
                    all32 = make_shift32_mult(mult, shift, m2) && all32;
                    s_m2[c] = m2;
                }
                cached_n_blk = n_blk;
                shift32 = named_barrier_and(2, EPI_THREADS, all32);
            }
            if (!dead) dead = !__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * ab, acc_phase, env, DEV_TIMEOUT_EPILOGUE));
            if (dead) continue;
            tc_fence_after();
            const int row = m_blk * 256 + (int)rank * BM + quarter * 32 + lane;
            int8_t* crow = p.C + (int64_t)row * p.ldc;
            const uint32_t t0 = tmem_base + ab * BN + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
            for (int ch = 0; ch < COLS_PER_GROUP / 32; ch++) {
                const int c0 = cgroup * COLS_PER_GROUP + ch * 32;
                const int n = n0 + c0;
                if (n >= p.N) break;
                int32_t v[32];
                tmem_ld_32x32(t0 + c0, v);
                tmem_ld_wait();
                if (p.raw) {
                    if (row < p.M) store_raw_chunk(p.D + (int64_t)row * p.ldd, n, p.N, p.c_vec_ok != 0, p.accumulate != 0, v);
                    continue;
                }
                uint32_t out[8];
                if (shift32) {
                    if (p.relu) epilogue_chunk_shift32<true>(v, s_bias, s_m2, c0, out);
                    else epilogue_chunk_shift32<false>(v, s_bias, s_m2, c0, out);
                } else {
                    epilogue_chunk(v, s_bias, s_lo, s_hi, s_mult, s_shift, s_rnd, c0, out);
                }
                if (row < p.M) store_row_chunk(crow, n, p.N, p.c_vec_ok != 0, out);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty0 + 8 * ab);   // this warp's share of the accumulator is free
            ab ^= 1;
            if (ab == 0) acc_phase ^= 1;
        }
    }

    tc_fence_before();
    cluster_sync_all();                                // neither CTA leaves or frees tensor memory while the other still works
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, L::TMEM_COLS);
    }
}

}  // namespace i8
