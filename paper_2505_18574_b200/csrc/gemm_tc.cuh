// Large-tile tensor path: persistent, warp-specialised int8 GEMM for sm_100a.
//
//   warp 0      producer : TMA loads of a 128 x 128-byte A tile and a BN x 128-byte B tile per ring slot
//   warp 1      MMA      : one thread issues tcgen05.mma kind::i8 (128 x BN x 32 per instruction) into one of two
//                          tensor-memory accumulators; the first instruction of a tile overwrites, the rest accumulate
//   warps 2..   epilogue : 4 or 8 warps read a finished accumulator (tcgen05.ld), apply bias/ReLU/scale/saturate,
//                          store int8
//
// The same kernel serves the convolution as an implicit GEMM (M = N*P*Q output pixels, N = filters,
// K = R*S*C): there the producer fetches A with TMA im2col loads straight from the NHWC activations, one
// load per filter tap and channel block, padding supplied by the out-of-bounds zero fill; no im2col
// matrix ever exists in memory.  A ring slot always holds 128 bytes of K per row, as 1, 2 or 4 sub-blocks
// of cb = 128, 64 or 32 bytes (cb = the channel block; plain GEMMs use one 128-byte block).
//
// TWO_SM = true runs the same roles on clusters of two CTAs that share one 256 x BN tile through
// tcgen05.mma.cta_group::2: each CTA holds 128 rows of A and BN / 2 rows of the B tile (a third less L2 and
// shared-memory traffic per product at BN = 256), the even CTA's MMA warp issues for both tensor cores, TMA loads of
// either CTA are counted on the even CTA's barriers, commits are multicast to both CTAs' barriers, and the odd CTA's
// epilogue warps arrive remotely on the even CTA's accumulator-free barrier.  No load uses cluster multicast.
//
// The roles map onto the decoupled load / execute / store controllers of the accelerator that the paper
// targets (Gemmini ISA description, Prompts appendix), and the two accumulators are the paper's
// accumulator double-buffering (Code Examples appendix, the optimised 12544x64x256 GEMM), so that the
// read-out of one tile overlaps the products of the next.
#pragma once
#include "epilogue.cuh"
#include "ptx.cuh"

namespace i8 {

constexpr int BM = 128;          // rows per tile = tensor-memory lanes
constexpr int BK = 128;          // bytes of K per ring slot = one 128-byte swizzle row
constexpr int UMMA_K = 32;       // K per tcgen05.mma for 8-bit operands

// Geometry of the K loop.  GEMM: cb = 128, nsub = 1, num_kblocks = ceil(K / 128).
// Convolution: cb = channel block, nsub = 128 / cb, num_kblocks = R * S * (C / cb).
struct KLoop {
    int cb, nsub, num_kblocks;
    int num_iters;                        // ring slots per tile = ceil(num_kblocks / nsub)
    int mmas_last;                        // tcgen05.mma instructions of a tile's last slot (1..4)
    int P, Q, S, cblocks;                 // convolution only: output extent, filter width, C / cb
    int stride_h, stride_w, pad_h, pad_w;
    uint32_t inv_pq, inv_q;               // floor(2^32 / (P*Q)) and floor(2^32 / Q) (0xffffffff for a divisor of 1)
    int b_resident;                       // the whole B operand of the (single) block column stays in shared memory
    // GEMM only: an operand stored with its M (A) or N (B) extent contiguous is fetched as K rows of 128 (64 for 64-wide
    // B tiles) contiguous bytes and consumed through an MN-major shared-memory descriptor: no transpose pass.  The maps
    // then have the contiguous extent as dimension 0 and K as dimension 1.
    int a_mn, b_mn;
};

// n / d for n < 2^31 with inv = floor(2^32 / d): the estimate is at most one too small.
__device__ __forceinline__ int fast_div(int n, int d, uint32_t inv) {
    int q = (int)__umulhi((uint32_t)n, inv);
    if (n - q * d >= d) ++q;
    return q;
}

// Two tile orders.  Grouped raster (sticky == 0): worker w takes tiles w, w + W, w + 2W, ... of a raster that walks
// group_m block rows at a time through all block columns (L2 reuse for the large problems).  Column-sticky (sticky != 0,
// chosen by the host for short-K problems with several tiles per worker): worker w owns block column w % n_tiles for the
// whole kernel and walks its rows slot, slot + S, slot + 2S, ... (S = workers of that column), so the per-channel
// epilogue constants are built once per CTA instead of once per tile.
struct TileSched {
    int m_tiles, n_tiles, num_tiles, group_m;
    int sticky, col_base, col_rem;        // column-sticky order: every column has col_base workers, the first col_rem one more
    // floor(2^32 / d) for the divisors below (0xffffffff for d == 1): a division costs a multiply and a fix-up instead
    // of the ~150-cycle software routine, which matters between the microsecond tiles of the small problems
    uint32_t inv_nt, inv_width, inv_gm, inv_step;     // n_tiles, group_m * n_tiles, group_m, number of workers
    uint32_t inv_last, inv_cb, inv_cb1;               // rows of the last (shorter) group, col_base, col_base + 1
    // one past the last tile index of worker w (tiles advance by `step` = number of workers)
    __device__ __forceinline__ int end_for(int w, int step) const {
        if (!sticky) return num_tiles;
        const int slot = fast_div(w, n_tiles, inv_nt), c = w - slot * n_tiles, S = col_base + (c < col_rem ? 1 : 0);
        const int count = slot < m_tiles ? fast_div(m_tiles - slot + S - 1, S, c < col_rem ? inv_cb1 : inv_cb) : 0;
        return w + count * step;
    }
    __device__ __forceinline__ void map(int tile, int w, int step, int& m_blk, int& n_blk) const {
        if (sticky) {
            const int it = fast_div(tile - w, step, inv_step);
            const int slot = fast_div(w, n_tiles, inv_nt);
            n_blk = w - slot * n_tiles;
            m_blk = slot + it * (col_base + (n_blk < col_rem ? 1 : 0));
            return;
        }
        if (n_tiles == 1) { m_blk = tile; n_blk = 0; return; }   // one block column: no divisions
        const int width = group_m * n_tiles;
        const int g = fast_div(tile, width, inv_width);
        const int first_m = g * group_m;
        const int gsz = min(m_tiles - first_m, group_m);
        const int local = tile - g * width;
        n_blk = gsz == group_m ? fast_div(local, group_m, inv_gm) : fast_div(local, gsz, inv_last);   // the last group may be shorter
        m_blk = first_m + local - n_blk * gsz;
    }
};

struct GemmTcParams {
    int8_t* C;
    int64_t ldc;
    const int32_t* bias;
    const int32_t* mult;
    const int32_t* shift;
    int per_channel, relu;
    int M, N, K;
    int c_vec_ok;               // C (or D) and its leading dimension are 16-byte aligned: full chunks go out as 16-byte stores
    int tma_store;              // wide tiles: int8 output leaves through shared memory and TMA stores (tmC is valid)
    int32_t* D;                 // raw read-out: the int32 accumulators themselves, no bias / activation / scale
    int64_t ldd;
    int raw, accumulate;        // raw != 0 selects D; accumulate != 0 adds to what D already holds
    TileSched sched;
    KLoop kl;
    // Independent problems of one shape in one launch (batch_mt != 0): the operands are read as matrices of stacked
    // problems, problem b starting a_rpp / b_rpp / c_rpp rows further in A / B / C, and the schedule's block rows run
    // over all problems (batch_mt block rows each).  Rows of a tile beyond M belong to the next problem in A and are
    // never stored; the bias of problem b starts bias_bs entries further.
    int batch_mt;
    uint32_t inv_bmt;           // floor(2^32 / batch_mt)
    int a_rpp, b_rpp;
    int64_t c_rpp, bias_bs;
    long long wait_limit_cycles;
    unsigned* dev_status;
};

template <int BN, int STAGES, bool TWO_SM = false>
struct TcSmem {
    static constexpr int B_ROWS = TWO_SM ? BN / 2 : BN;        // a CTA of a pair holds half of the tile's B rows
    static constexpr int A_BYTES = BM * BK;
    static constexpr int B_BYTES = B_ROWS * BK;
    static constexpr int OFF_A = 0;
    static constexpr int OFF_B = OFF_A + STAGES * A_BYTES;
    static constexpr int OFF_CONST = OFF_B + STAGES * B_BYTES;       // 7 int32[BN] arrays and one int64[BN] array of per-channel constants
    static constexpr int OFF_BAR = OFF_CONST + 9 * BN * 4;           // full[S], empty[S], acc_full[2], acc_empty[2], b_resident
    static constexpr int OFF_MISC = OFF_BAR + (2 * STAGES + 5) * 8;  // tensor-memory base, stop flag
    // read-out staging of the wide tiles: every epilogue warp collects 32 rows x 64 output bytes (64-byte swizzle) and one
    // lane hands them to the TMA engine: the 32 scattered row segments cost the load/store pipe nothing
    static constexpr int STAGE_WARP_BYTES = 32 * 64;
    static constexpr int OFF_STAGE = (OFF_MISC + 16 + 1023) / 1024 * 1024;
    static constexpr int TOTAL = BN >= 128 ? OFF_STAGE + 8 * STAGE_WARP_BYTES : OFF_MISC + 16;
    static constexpr int DYN_BYTES = TOTAL + 1024;                   // slack to align the base to 1024 bytes
    static constexpr int TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;      // BN in {64,128,256}: a power of two
};

// Epilogue arithmetic for one 32-column chunk held in v[]; column constants come from shared memory.
__device__ __forceinline__ void epilogue_chunk(const int32_t (&v)[32], const int32_t* s_bias, const int32_t* s_lo,
                                               const int32_t* s_hi, const int32_t* s_mult, const int32_t* s_shift,
                                               const int32_t* s_rnd, int c0, uint32_t (&out)[8]) {
#pragma unroll
    for (int j = 0; j < 8; j++) {
        const int4 bi = *reinterpret_cast<const int4*>(s_bias + c0 + 4 * j);
        const int4 lo = *reinterpret_cast<const int4*>(s_lo + c0 + 4 * j);
        const int4 hi = *reinterpret_cast<const int4*>(s_hi + c0 + 4 * j);
        const int4 mu = *reinterpret_cast<const int4*>(s_mult + c0 + 4 * j);
        const int4 sh = *reinterpret_cast<const int4*>(s_shift + c0 + 4 * j);
        const int4 rn = *reinterpret_cast<const int4*>(s_rnd + c0 + 4 * j);
        const int32_t r0 = requant_fast(v[4 * j + 0], bi.x, lo.x, hi.x, mu.x, sh.x, rn.x);
        const int32_t r1 = requant_fast(v[4 * j + 1], bi.y, lo.y, hi.y, mu.y, sh.y, rn.y);
        const int32_t r2 = requant_fast(v[4 * j + 2], bi.z, lo.z, hi.z, mu.z, sh.z, rn.z);
        const int32_t r3 = requant_fast(v[4 * j + 3], bi.w, lo.w, hi.w, mu.w, sh.w, rn.w);
        out[j] = pack_sat4(r0, r1, r2, r3);
    }
}

// Same chunk in the shift-32 form with constants from shared memory: half a 16-byte load, one add, at most one
// max and one widening multiply-add per output.
template <bool RELU>
__device__ __forceinline__ void epilogue_chunk_shift32(const int32_t (&v)[32], const int32_t* s_bias, const int32_t* s_m2,
                                                       int c0, uint32_t (&out)[8]) {
#pragma unroll
    for (int j = 0; j < 8; j++) {
        const int4 bi = *reinterpret_cast<const int4*>(s_bias + c0 + 4 * j);
        const int4 m2 = *reinterpret_cast<const int4*>(s_m2 + c0 + 4 * j);
        out[j] = pack_sat4(requant_shift32<RELU>(v[4 * j + 0], bi.x, m2.x), requant_shift32<RELU>(v[4 * j + 1], bi.y, m2.y),
                           requant_shift32<RELU>(v[4 * j + 2], bi.z, m2.z), requant_shift32<RELU>(v[4 * j + 3], bi.w, m2.w));
    }
}

// Folded form with the bias added explicitly: two words per channel from shared memory instead of three (a 16-byte
// shared-memory broadcast costs four wavefronts, and eight epilogue warps each fetch every channel's constants).
template <bool RELU>
__device__ __forceinline__ void epilogue_chunk_fold_add(const int32_t (&v)[32], const int32_t* s_bias, const int32_t* s_m2, int c0,
                                                        uint32_t (&out)[8]) {
#pragma unroll
    for (int j = 0; j < 8; j++) {
        const int4 bi = *reinterpret_cast<const int4*>(s_bias + c0 + 4 * j);
        const int4 m2 = *reinterpret_cast<const int4*>(s_m2 + c0 + 4 * j);
        const uint32_t pk = pack_sat4(requant_fold(v[4 * j + 0] + bi.x, m2.x, 1ll << 31), requant_fold(v[4 * j + 1] + bi.y, m2.y, 1ll << 31),
                                      requant_fold(v[4 * j + 2] + bi.z, m2.z, 1ll << 31), requant_fold(v[4 * j + 3] + bi.w, m2.w, 1ll << 31));
        out[j] = RELU ? relu_s8x4(pk) : pk;
    }
}
// Folded form, bias added explicitly, constants in registers (two words per channel).
template <bool RELU>
__device__ __forceinline__ void epilogue_chunk_fold_add_regs(const int32_t (&v)[32], const int32_t (&rb)[32], const int32_t (&rm)[32],
                                                             uint32_t (&out)[8]) {
#pragma unroll
    for (int j = 0; j < 8; j++) {
        const uint32_t pk = pack_sat4(requant_fold(v[4 * j + 0] + rb[4 * j + 0], rm[4 * j + 0], 1ll << 31), requant_fold(v[4 * j + 1] + rb[4 * j + 1], rm[4 * j + 1], 1ll << 31),
                                      requant_fold(v[4 * j + 2] + rb[4 * j + 2], rm[4 * j + 2], 1ll << 31), requant_fold(v[4 * j + 3] + rb[4 * j + 3], rm[4 * j + 3], 1ll << 31));
        out[j] = RELU ? relu_s8x4(pk) : pk;
    }
}

// Store one thread's 32 output bytes (columns n .. n+31 of one row).
__device__ __forceinline__ void store_row_chunk(int8_t* crow, int n, int N, bool vec_ok, const uint32_t (&out)[8]) {
    if (vec_ok && n + 32 <= N) {
        uint4* dst = reinterpret_cast<uint4*>(crow + n);
        dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
        dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
    } else {
#pragma unroll
        for (int j = 0; j < 32; j++)
            if (n + j < N) crow[n + j] = (int8_t)((out[j >> 2] >> (8 * (j & 3))) & 0xff);
    }
}

// Raw read-out of one thread's 32 accumulators (columns n .. n+31 of one row), optionally added to the destination.
__device__ __forceinline__ void store_raw_chunk(int32_t* drow, int n, int N, bool vec_ok, bool accumulate, const int32_t (&v)[32]) {
    if (vec_ok && n + 32 <= N) {
        int4* dst = reinterpret_cast<int4*>(drow + n);
#pragma unroll
        for (int j = 0; j < 8; j++) {
            int4 o = make_int4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            if (accumulate) { const int4 e = dst[j]; o.x += e.x; o.y += e.y; o.z += e.z; o.w += e.w; }
            dst[j] = o;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 32; j++)
            if (n + j < N) drow[n + j] = accumulate ? drow[n + j] + v[j] : v[j];
    }
}

template <int BN, int STAGES, bool CONV, int EPI_WARPS, int NPROD, bool TWO_SM>
__global__ void __launch_bounds__(32 * (1 + NPROD) + 32 * EPI_WARPS, 1)
gemm_i8_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmC, const GemmTcParams p) {
    using L = TcSmem<BN, STAGES, TWO_SM>;
    constexpr int EPI_THREADS = 32 * EPI_WARPS;
    constexpr int TILE_M = TWO_SM ? 2 * BM : BM;       // rows of one output tile (a CTA pair shares a 256-row tile)
    constexpr int B_ROWS = L::B_ROWS;
    constexpr int NTHREADS = 32 * (1 + NPROD) + EPI_THREADS;
    constexpr int PROD2_WARP = 2 + EPI_WARPS;         // the optional second producer is the last warp
    static_assert(NPROD == 1 || NPROD == 2, "one or two producer warps");
    static_assert(STAGES % 2 == 0, "two producers alternate ring slots");
    constexpr int COL_GROUPS = EPI_WARPS / 4;          // warps sharing a lane quarter split the columns
    constexpr int COLS_PER_GROUP = BN / COL_GROUPS;
    static_assert(EPI_WARPS == 4 || EPI_WARPS == 8, "4 or 8 epilogue warps");
    static_assert(COLS_PER_GROUP % 32 == 0, "column split must keep 32-column chunks");

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
    long long* s_c64 = reinterpret_cast<long long*>(s_rnd + BN);     // folded form: bias * m2 + 2^31 (8-byte aligned: BN is even)
    const uint32_t bar_full = sbase + L::OFF_BAR;
    const uint32_t bar_empty = bar_full + STAGES * 8;
    const uint32_t bar_acc_full = bar_empty + STAGES * 8;
    const uint32_t bar_acc_empty = bar_acc_full + 2 * 8;
    const uint32_t bar_bres = bar_acc_empty + 2 * 8;
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + L::OFF_MISC);
    volatile int* s_stop = reinterpret_cast<volatile int*>(smem + L::OFF_MISC + 4);

    // broadcast from lane 0 so the compiler can treat the role index as warp-uniform
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    const WaitEnv env{s_stop, p.dev_status, p.wait_limit_cycles};
    // CTA pairs: rank 0 (even CTA) issues the MMAs; its full / accumulator-free / resident-B barriers serve both CTAs
    const uint32_t rank = TWO_SM ? cluster_ctarank() : 0u;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(bar_acc_full + 8 * b, 1);
            // one-SM: every epilogue thread arrives; pair: one lane of every epilogue warp of both CTAs
            mbar_init(bar_acc_empty + 8 * b, TWO_SM ? 2 * EPI_WARPS : EPI_THREADS);
        }
        mbar_init(bar_bres, 1);
        *s_stop = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        if (TWO_SM) {
            tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(s_tmem)), L::TMEM_COLS);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(const_cast<uint32_t*>(s_tmem)), L::TMEM_COLS);
            tmem_relinquish();
        }
    }
    if (warp == 0 && lane == 0) {
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    // The next kernel of the stream may be scheduled from here on; this one goes on with set-up that touches only shared
    // and tensor memory, and waits for its own predecessor right before the roles start (below).
    grid_launch_dependents();
    // Set-up barrier.  The producer warp initialised the mbarriers itself and needs nothing from the others, so it
    // only signals and starts loading at once; everybody else waits for the barriers and the tensor-memory address.
    uint32_t tmem_base = 0;
    if (TWO_SM) {
        // both CTAs' barriers must exist before anything remote touches them
        tc_fence_before();
        cluster_sync_all();
        tc_fence_after();
        tmem_base = __shfl_sync(0xffffffffu, *s_tmem, 0);
    } else if (warp == 0) {
        __syncwarp();
        named_barrier_arrive(15, NTHREADS);
    } else if (NPROD == 2 && warp == PROD2_WARP) {
        named_barrier(15, NTHREADS);                      // needs the initialised barriers, nothing else
    } else {
        tc_fence_before();
        named_barrier(15, NTHREADS);
        tc_fence_after();
        tmem_base = __shfl_sync(0xffffffffu, *s_tmem, 0);   // same value in every lane, known uniform
    }

    const TileSched sched = p.sched;
    const KLoop kl = p.kl;
    const uint32_t a_sub_bytes = BM * kl.cb, b_sub_bytes = B_ROWS * kl.cb;
    // persistent schedule: CTA (or CTA pair) w takes tiles w, w + W, w + 2W, ...
    const int first_tile = TWO_SM ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int tile_step = TWO_SM ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    const int tile_end = sched.end_for(first_tile, tile_step);
    // barriers of the even CTA, as seen from this CTA (its own in the one-SM kernel)
    const uint32_t full0 = TWO_SM ? map_to_cta(bar_full, 0) : bar_full;
    const uint32_t bres0 = TWO_SM ? map_to_cta(bar_bres, 0) : bar_bres;
    const uint32_t acc_empty0 = TWO_SM ? map_to_cta(bar_acc_empty, 0) : bar_acc_empty;
    const uint32_t tx_mult = TWO_SM ? 2u : 1u;         // the even CTA's barriers count both CTAs' bytes
    // Global memory is read and written from here on: everything the preceding kernel wrote must be visible.
    grid_dependency_wait();

    if (warp == 0 || (NPROD == 2 && warp == PROD2_WARP)) {
        // ------------------------------------------------------------------ producer (whole warp loops, one lane issues)
        // With two producer warps, warp 0 fills the even ring slots and the last warp the odd ones; both walk the
        // same sequence of tiles and slots and skip the slots that are not theirs.
        const int pid = warp == 0 ? 0 : 1;
        int stage = 0;
        uint32_t phase = 0, issued = 0, issued_phase = 0;
        bool ok = true, first_pass = true;
        const bool leader = elect_one();
        const bool bres = kl.b_resident != 0;
        if (bres && pid == 0 && first_tile < tile_end && leader) {
            // the paper's "keep B resident" step: the whole (small) B operand is fetched once per CTA into the
            // region the ring would otherwise use for B, and only A streams
            if (rank == 0) mbar_expect_tx(bar_bres, tx_mult * kl.num_kblocks * b_sub_bytes);
            for (int kb = 0; kb < kl.num_kblocks; kb++) {
                if (TWO_SM) tma_load_2d_pair(sB + kb * b_sub_bytes, &tmB, bres0, kb * kl.cb, (int)rank * B_ROWS);
                else tma_load_2d(sB + kb * b_sub_bytes, &tmB, bar_bres, kb * kl.cb, 0);
            }
        }
        const uint32_t stage_tx = a_sub_bytes + (bres ? 0u : b_sub_bytes);
        for (int tile = first_tile; ok && tile < tile_end; tile += tile_step) {
            int m_blk, n_blk;
            sched.map(tile, first_tile, tile_step, m_blk, n_blk);
            int prob = 0;                                               // which of the stacked problems
            if (p.batch_mt) { prob = fast_div(m_blk, p.batch_mt, p.inv_bmt); m_blk -= prob * p.batch_mt; }
            const int row_a = prob * p.a_rpp + m_blk * TILE_M + (int)rank * BM;   // this CTA's first A row (output row / pixel)
            // this CTA's first B row (output column); a stacked problem starts b_rpp rows further: rows of N for K-major B,
            // rows of K for MN-major B (where a ragged last K block then reads the next problem's rows: they meet the
            // zeros that A's own K edge is filled with)
            const int b_mn_now = !CONV && kl.b_mn;
            const int row_b = (b_mn_now ? 0 : prob * p.b_rpp) + n_blk * BN + (int)rank * B_ROWS;
            const int k_off_b = b_mn_now ? prob * p.b_rpp : 0;
            int w0 = 0, h0 = 0, img = 0;
            if (CONV) {
                // first output pixel of the tile -> position of filter tap (0,0) in the input image
                const int m0 = row_a;
                const int pq = kl.P * kl.Q;
                img = fast_div(m0, pq, kl.inv_pq);
                const int rem = m0 - img * pq;
                const int op = fast_div(rem, kl.Q, kl.inv_q), oq = rem - op * kl.Q;
                h0 = op * kl.stride_h - kl.pad_h;
                w0 = oq * kl.stride_w - kl.pad_w;
            }
            int c_idx = 0, fs = 0, fr = 0;      // convolution: channel block, filter column, filter row
            for (int kbi = 0; kbi < kl.num_kblocks;) {
                const int nb = min(kl.nsub, kl.num_kblocks - kbi);
                if (NPROD == 2 && (stage & 1) != pid) {
                    // the other producer's slot: only keep the tap / channel counters in step
                    for (int j = 0; j < nb; j++, kbi++)
                        if (CONV && ++c_idx == kl.cblocks) { c_idx = 0; if (++fs == kl.S) { fs = 0; ++fr; } }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; first_pass = false; }
                    continue;
                }
                // on the first pass over the ring every slot is free: nothing to wait for
                if (!first_pass && !mbar_wait_warp(bar_empty + 8 * stage, phase ^ 1, env, DEV_TIMEOUT_PRODUCER)) { ok = false; break; }
                const uint32_t full = full0 + 8 * stage;
                if (leader && rank == 0) mbar_expect_tx(bar_full + 8 * stage, tx_mult * nb * stage_tx);
                for (int j = 0; j < nb; j++, kbi++) {
                    const uint32_t dstA = sA + stage * L::A_BYTES + j * a_sub_bytes;
                    const uint32_t dstB = sB + stage * L::B_BYTES + j * b_sub_bytes;
                    if (CONV) {
                        if (leader) {
                            if (TWO_SM) tma_load_im2col_4d_pair(dstA, &tmA, full, c_idx * kl.cb, w0, h0, img, (uint16_t)fs, (uint16_t)fr);
                            else tma_load_im2col_4d(dstA, &tmA, full, c_idx * kl.cb, w0, h0, img, (uint16_t)fs, (uint16_t)fr);
                        }
                        if (++c_idx == kl.cblocks) { c_idx = 0; if (++fs == kl.S) { fs = 0; ++fr; } }
                    } else if (leader) {
                        // K-major: (k, row); MN-major: (row, k), the 128 K rows of the slot 128 bytes apart
                        const int ax = kl.a_mn ? row_a : kbi * BK, ay = kl.a_mn ? kbi * BK : row_a;
                        if (TWO_SM) tma_load_2d_pair(dstA, &tmA, full, ax, ay);
                        else tma_load_2d(dstA, &tmA, full, ax, ay);
                    }
                    if (leader && !bres) {
                        if (!CONV && kl.b_mn) {
                            // one box of K rows per 128 columns of the tile (a 64-wide tile: one box of 64-byte rows)
                            constexpr int NBOX = B_ROWS > 128 ? B_ROWS / 128 : 1;
#pragma unroll
                            for (int h = 0; h < NBOX; h++) {
                                if (TWO_SM) tma_load_2d_pair(dstB + h * (128 * BK), &tmB, full, row_b + h * 128, k_off_b + kbi * BK);
                                else tma_load_2d(dstB + h * (128 * BK), &tmB, full, row_b + h * 128, k_off_b + kbi * BK);
                            }
                        } else {
                            if (TWO_SM) tma_load_2d_pair(dstB, &tmB, full, kbi * kl.cb, row_b);
                            else tma_load_2d(dstB, &tmB, full, kbi * kl.cb, row_b);
                        }
                    }
                }
                issued |= 1u << stage;
                issued_phase = (issued_phase & ~(1u << stage)) | (phase << stage);
                if (++stage == STAGES) { stage = 0; phase ^= 1; first_pass = false; }
            }
        }
        if (*s_stop && rank == 0) {
            // stopping early: let every copy this warp started land before the CTA retires (in a pair the even CTA's
            // barriers also count the odd CTA's copies, and the closing cluster barrier keeps the odd CTA alive meanwhile)
            if (bres && pid == 0 && first_tile < tile_end && !mbar_wait_drain(bar_bres, 0, p.wait_limit_cycles))
                atomicCAS(p.dev_status, 0u, (unsigned)DEV_TIMEOUT_DRAIN);
            for (int s = 0; s < STAGES; s++)
                if (issued & (1u << s))
                    if (!mbar_wait_drain(bar_full + 8 * s, (issued_phase >> s) & 1u, p.wait_limit_cycles))
                        atomicCAS(p.dev_status, 0u, (unsigned)DEV_TIMEOUT_DRAIN);
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (whole warp loops, one lane issues)
        const uint32_t idesc = make_idesc_i8(TILE_M, BN, kl.a_mn, kl.b_mn);   // a pair's instruction spans both CTAs' rows
        // K-major operands: rows cb bytes apart, swizzled over cb bytes, 8-row groups 8*cb bytes apart;
        // a 32-byte step along K inside a swizzle row is a plain address offset.
        const uint64_t swz = kl.cb == 128 ? SWZ_128B : (kl.cb == 64 ? SWZ_64B : SWZ_32B);
        const uint64_t desc_k = make_smem_desc(0, 16, 8 * kl.cb, swz);   // everything but the start address
        // MN-major operands: K rows of `mnw` contiguous bytes (128; 64 for a 64-wide B tile), swizzled over mnw bytes;
        // 8 K rows are one group (stride offset 8 * mnw), the next block of mnw columns starts one whole box further
        // (leading offset 128 rows * mnw), and 32 of K is 32 rows.
        constexpr int B_MNW = B_ROWS >= 128 ? 128 : 64;
        const uint64_t desc_hi_a = kl.a_mn ? make_smem_desc(0, 128 * 128, 8 * 128, SWZ_128B) : desc_k;
        const uint64_t desc_hi_b = (!CONV && kl.b_mn) ? make_smem_desc(0, 128 * B_MNW, 8 * B_MNW, B_MNW == 128 ? SWZ_128B : SWZ_64B) : desc_k;
        const bool leader = elect_one();
        // A full ring slot always takes BK / 32 = 4 instructions; their operand offsets (in 16-byte descriptor
        // units) inside the slot depend only on the sub-block geometry.
        const int per_sub = kl.cb / UMMA_K;
        uint32_t offA[4], offB[4];
#pragma unroll
        for (int i = 0; i < 4; i++) {
            const int sub = i / per_sub, k = i - sub * per_sub;
            offA[i] = (kl.a_mn ? i * UMMA_K * 128 : sub * a_sub_bytes + k * UMMA_K) >> 4;
            offB[i] = ((!CONV && kl.b_mn) ? i * UMMA_K * B_MNW : sub * b_sub_bytes + k * UMMA_K) >> 4;
        }
        const uint32_t a_base = (sA & 0x3FFFFu) >> 4, b_base = (sB & 0x3FFFFu) >> 4;
        int stage = 0, ab = 0;
        uint32_t phase = 0, acc_phase = 0;
        bool ready = false;                              // the slot (stage, phase) is already known to be full
        bool ok = true;
        const bool bres = kl.b_resident != 0;
        const uint32_t b_iter_units = (kl.nsub * b_sub_bytes) >> 4;   // resident B: descriptor units per ring slot's worth of K
        if (rank != 0) ok = false;                       // in a pair only the even CTA issues
        if (ok && bres && first_tile < tile_end) ok = mbar_wait_warp(bar_bres, 0, env, DEV_TIMEOUT_MMA_FULL);
        for (int tile = first_tile; ok && tile < tile_end; tile += tile_step) {
            if (!mbar_wait_warp(bar_acc_empty + 8 * ab, acc_phase ^ 1, env, DEV_TIMEOUT_MMA_ACC)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + ab * BN;
            for (int it = 0; it < kl.num_iters; it++) {
                if (!ready && !mbar_wait_warp(bar_full + 8 * stage, phase, env, DEV_TIMEOUT_MMA_FULL)) { ok = false; break; }
                tc_fence_after();
                // poll the next slot now; its answer is only needed after this slot's instructions are issued
                int nstage = stage + 1;
                uint32_t nphase = phase;
                if (nstage == STAGES) { nstage = 0; nphase ^= 1; }
                const bool peek = mbar_test_wait(bar_full + 8 * nstage, nphase);
                if (leader) {
                    const int nm = it == kl.num_iters - 1 ? kl.mmas_last : 4;
                    const uint32_t a0 = a_base + stage * (L::A_BYTES >> 4);
                    const uint32_t b0 = b_base + (bres ? it * b_iter_units : stage * (L::B_BYTES >> 4));
#pragma unroll
                    for (int i = 0; i < 4; i++)
                        if (i < nm) {
                            if (TWO_SM) mma_i8_ss_pair(d_tmem, desc_hi_a | (uint64_t)(a0 + offA[i]), desc_hi_b | (uint64_t)(b0 + offB[i]), idesc,
                                                       (it | i) != 0 ? 1u : 0u);
                            else mma_i8_ss(d_tmem, desc_hi_a | (uint64_t)(a0 + offA[i]), desc_hi_b | (uint64_t)(b0 + offB[i]), idesc,
                                           (it | i) != 0 ? 1u : 0u);
                        }
                    // slot reusable once these MMAs have read it (in a pair: in both CTAs)
                    if (TWO_SM) tc_commit_pair(bar_empty + 8 * stage);
                    else tc_commit(bar_empty + 8 * stage);
                }
                ready = __all_sync(0xffffffffu, peek);
                stage = nstage;
                phase = nphase;
            }
            if (!ok) break;
            if (leader) {                                    // accumulator complete (both halves in a pair)
                if (TWO_SM) tc_commit_pair(bar_acc_full + 8 * ab);
                else tc_commit(bar_acc_full + 8 * ab);
            }
            ab ^= 1;
            if (ab == 0) acc_phase ^= 1;
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue
        const int etid = threadIdx.x - 64;
        const int quarter = warp & 3;                   // a warp may only read lanes 32*(warp%4) .. +31
        const int cgroup = (warp - 2) >> 2;             // which share of the columns this warp handles
        int ab = 0, cached_n_blk = -1;
        bool shift32 = false;                           // every channel of the cached block admits the shift-32 form
        bool fold = false;                              // ... and the folded form (under ReLU: no negative multiplier)
        constexpr bool ONE_CHUNK = COLS_PER_GROUP == 32;
        // register copy of the constants (ONE_CHUNK only: 64-wide tiles): no shared-memory broadcast per output.  (128-wide
        // tiles on 16 epilogue warps would qualify too; measured on the 1x1 layer with 2048 filters that instance is a third
        // slower: 96 registers per thread spill, and its direct row stores replace the staged TMA stores.)
        int32_t rm[ONE_CHUNK ? 32 : 1], rb[ONE_CHUNK ? 32 : 1];
        uint32_t acc_phase = 0;
        bool dead = false;
        for (int tile = first_tile; tile < tile_end; tile += tile_step) {
            int m_blk, n_blk;
            sched.map(tile, first_tile, tile_step, m_blk, n_blk);
            int prob = 0;
            if (p.batch_mt) { prob = fast_div(m_blk, p.batch_mt, p.inv_bmt); m_blk -= prob * p.batch_mt; }
            const int n0 = n_blk * BN;
            const int col_key = p.bias_bs ? n_blk + prob * sched.n_tiles : n_blk;   // a per-problem bias: new constants per problem
            if (col_key != cached_n_blk) {
                // new block column: rebuild the per-channel constants (before waiting, so this overlaps the main loop)
                named_barrier(1, EPI_THREADS);            // nobody still reads the previous column's constants
                bool all32 = true, allfold = true;
                for (int c = etid; c < BN; c += EPI_THREADS) {
                    const int n = n0 + c;
                    int32_t bias = 0, mult = 0, shift = 0;
                    if (n < p.N && !p.raw) {
                        bias = p.bias ? p.bias[(int64_t)prob * p.bias_bs + n] : 0;
                        mult = p.mult[p.per_channel ? n : 0];
                        shift = p.shift[p.per_channel ? n : 0];
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
                cached_n_blk = col_key;
                shift32 = named_barrier_and(2, EPI_THREADS, all32);
                fold = named_barrier_and(3, EPI_THREADS, allfold);
                if constexpr (ONE_CHUNK) if (fold) {
                    // this warp's 32 columns are the same for every tile of the block column: keep them in registers
#pragma unroll
                    for (int j = 0; j < 32; j++) { rm[j] = s_m2[cgroup * 32 + j]; rb[j] = s_bias[cgroup * 32 + j]; }
                }
            }
            // A warp whose wait expired stays in the loop without touching the accumulators, so that the barriers
            // above still see every warp; the stop flag it raised ends the other roles.
            if (!dead) dead = !__all_sync(0xffffffffu, mbar_wait(bar_acc_full + 8 * ab, acc_phase, env, DEV_TIMEOUT_EPILOGUE));
            if (dead) continue;
            tc_fence_after();
            const int row = m_blk * TILE_M + (int)rank * BM + quarter * 32 + lane;
            int8_t* crow = p.C + ((int64_t)prob * p.c_rpp + row) * p.ldc;
            const uint32_t t0 = tmem_base + ab * BN + ((uint32_t)(quarter * 32) << 16);
            // staging buffer of this warp: row r holds four 16-byte units, unit u at position u ^ ((r >> 1) & 3) (the
            // 64-byte TMA swizzle, which also keeps the row-wise 16-byte writes free of bank conflicts)
            const uint32_t stage_w = sbase + L::OFF_STAGE + (warp - 2) * L::STAGE_WARP_BYTES;
            const bool staged = !ONE_CHUNK && p.tma_store != 0;
#pragma unroll 1
            for (int ch = 0; ch < COLS_PER_GROUP / 32; ch++) {
                const int c0 = cgroup * COLS_PER_GROUP + ch * 32;
                const int n = n0 + c0;
                if (n >= p.N) break;
                int32_t v[32];
                tmem_ld_32x32(t0 + c0, v);
                tmem_ld_wait();
                if (p.raw) {
                    // the accumulator read as accumulator-type data (Gemmini's unscaled read-out), optionally
                    // accumulated on top of the destination (its accumulate-on-write mode)
                    if (row < p.M) store_raw_chunk(p.D + (int64_t)row * p.ldd, n, p.N, p.c_vec_ok != 0, p.accumulate != 0, v);
                    continue;
                }
                uint32_t out[8];
                if (fold) {
                    if constexpr (ONE_CHUNK) {
                        if (p.relu) epilogue_chunk_fold_add_regs<true>(v, rb, rm, out);
                        else epilogue_chunk_fold_add_regs<false>(v, rb, rm, out);
                    } else {
                        if (p.relu) epilogue_chunk_fold_add<true>(v, s_bias, s_m2, c0, out);
                        else epilogue_chunk_fold_add<false>(v, s_bias, s_m2, c0, out);
                    }
                } else if (shift32) {
                    // ReLU with a negative multiplier somewhere in the block column: ReLU must stay ahead of the scale
                    if (p.relu) epilogue_chunk_shift32<true>(v, s_bias, s_m2, c0, out);
                    else epilogue_chunk_shift32<false>(v, s_bias, s_m2, c0, out);
                } else {
                    epilogue_chunk(v, s_bias, s_lo, s_hi, s_mult, s_shift, s_rnd, c0, out);
                }
                if constexpr (!ONE_CHUNK) {
                    if (staged) {
                        if ((ch & 1) == 0) {
                            // the previous pair's copy must have read the buffer before it is refilled
                            if (lane == 0) tma_store_wait_read();
                            __syncwarp();
                        }
                        const uint32_t srow = stage_w + lane * 64;
                        const uint32_t sw = (lane >> 1) & 3, u0 = 2 * (ch & 1);
                        st_shared_v4(srow + ((u0 ^ sw) << 4), out[0], out[1], out[2], out[3]);
                        st_shared_v4(srow + (((u0 + 1) ^ sw) << 4), out[4], out[5], out[6], out[7]);
                        // a pair is complete after its second chunk, or when the block column ends after the first
                        if ((ch & 1) || n + 32 >= p.N) {
                            fence_proxy_async_smem();
                            __syncwarp();
                            // rows beyond M and columns beyond N are clipped by the copy engine (stale bytes of an
                            // unwritten second half only ever fall there)
                            const int y0 = m_blk * TILE_M + (int)rank * BM + quarter * 32;
                            if (lane == 0 && y0 < p.M) {
                                tma_store_2d(&tmC, stage_w, n - 32 * (ch & 1), y0);
                                tma_store_commit();
                            }
                        }
                        continue;
                    }
                }
                if (row < p.M) store_row_chunk(crow, n, p.N, p.c_vec_ok != 0, out);
            }
            tc_fence_before();
            if (TWO_SM) {
                // one lane per warp tells the even CTA that this warp's share of the accumulator is free
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(acc_empty0 + 8 * ab);
            } else {
                mbar_arrive(bar_acc_empty + 8 * ab);
            }
            ab ^= 1;
            if (ab == 0) acc_phase ^= 1;
        }
    }

    if (warp >= 2 && warp < 2 + EPI_WARPS && lane == 0) tma_store_wait_all();   // this lane's output copies are complete
    tc_fence_before();
    if (TWO_SM) {
        cluster_sync_all();        // neither CTA leaves or frees tensor memory while the other still works
        if (warp == 1) {
            tc_fence_after();
            tmem_dealloc_pair(tmem_base, L::TMEM_COLS);
        }
    } else {
        __syncthreads();
        if (warp == 1) {
            tc_fence_after();
            tmem_dealloc(tmem_base, L::TMEM_COLS);
        }
    }
}

}  // namespace i8
