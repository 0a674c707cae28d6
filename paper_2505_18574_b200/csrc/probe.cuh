// Issue-rate probe of tcgen05.mma kind::i8: the measured int8 tensor peak that roofline fractions are quoted against.
//
// Every CTA (one per SM) fills two shared-memory tiles with pseudo-random bytes, then one thread issues `reps`
// instructions of 128 x N x 32 back to back on those resident operands (128-byte-swizzled K-major tiles, the layout of
// the GEMM kernel's ring slots) into two alternating tensor-memory accumulators and waits for the last one to finish.
// Nothing is loaded from or stored to global memory inside the timed part, so the time is what the tensor core itself
// needs: the ceiling any kernel built on this instruction can reach at the clock the GPU sustains under that load.
// Timing only: the products are never read.
#pragma once
#include "ptx.cuh"

namespace i8 {

constexpr int PROBE_A_BYTES = 128 * 128;            // 128 rows x 128 bytes of K
constexpr int PROBE_B_BYTES = 256 * 128;            // up to 256 rows x 128 bytes of K
constexpr int PROBE_THREADS = 128;
// one CTA per SM: ask for more than half of an SM's shared memory
constexpr int PROBE_SMEM = 120 * 1024;
static_assert(PROBE_A_BYTES + PROBE_B_BYTES + 64 + 1024 <= PROBE_SMEM, "operands and barrier fit the allocation");

struct MmaProbeParams {
    int n;                        // instruction width: 16 .. 256, a multiple of 16
    int reps;                     // instructions per CTA, a multiple of 64
    unsigned long long* out;      // [gridDim.x][4]: issue cycles, cycles until complete, ns until complete, SM id
    long long wait_limit_cycles;
    unsigned* dev_status;
};

__global__ void __launch_bounds__(PROBE_THREADS, 1) mma_issue_probe_kernel(const MmaProbeParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = (1024u - (raw & 1023u)) & 1023u;
    uint8_t* smem = smem_raw + pad;
    const uint32_t sbase = raw + pad, sA = sbase, sB = sbase + PROBE_A_BYTES;
    const uint32_t bar_done = sbase + PROBE_A_BYTES + PROBE_B_BYTES;
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + PROBE_A_BYTES + PROBE_B_BYTES + 16);
    volatile int* s_stop = reinterpret_cast<volatile int*>(smem + PROBE_A_BYTES + PROBE_B_BYTES + 20);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // operands: every byte of both tiles gets a pseudo-random value (all-zero operands would draw less power)
    {
        uint32_t x = 0x9E3779B9u * (blockIdx.x * PROBE_THREADS + threadIdx.x + 1);
        uint32_t* w = reinterpret_cast<uint32_t*>(smem);
        for (int i = threadIdx.x; i < (PROBE_A_BYTES + PROBE_B_BYTES) / 4; i += PROBE_THREADS) {
            x ^= x << 13; x ^= x >> 17; x ^= x << 5;
            w[i] = x;
        }
    }
    if (threadIdx.x == 0) {
        mbar_init(bar_done, 1);
        *s_stop = 0;
        fence_barrier_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(s_tmem)), 512);
        tmem_relinquish();
    }
    fence_proxy_async_smem();            // the tensor core reads the tiles through the async proxy
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem;
    const WaitEnv env{s_stop, p.dev_status, p.wait_limit_cycles};

    if (warp == 0) {
        long long t0 = 0, t1 = 0;
        unsigned long long ns0 = 0;
        if (lane == 0) {
            // K-major, 128-byte swizzle: rows 128 bytes apart, 8-row groups 1024 bytes apart; the four 32-byte K steps of
            // a row are plain address offsets.  Furthest byte read: A 127 * 128 + 96 + 32 = 16384 = PROBE_A_BYTES,
            // B (n - 1) * 128 + 128 <= PROBE_B_BYTES for n <= 256 (checked on the host).
            const uint64_t hi = make_smem_desc(0, 16, 1024, SWZ_128B);
            const uint32_t a0 = (sA & 0x3FFFFu) >> 4, b0 = (sB & 0x3FFFFu) >> 4;
            const uint32_t idesc = make_idesc_i8(128, p.n, 0, 0);
            ns0 = globaltimer_ns();
            t0 = clock64();
            for (int i = 0; i < p.reps; i += 64) {
                const uint32_t d = tmem_base + (((i >> 6) & 1) ? 256u : 0u);
#pragma unroll
                for (int j = 0; j < 64; j++) {
                    const uint32_t k = (uint32_t)(j & 3) * 2;                 // 32 bytes = 2 descriptor units
                    mma_i8_ss(d, hi | (uint64_t)(a0 + k), hi | (uint64_t)(b0 + k), idesc, j != 0 ? 1u : 0u);
                }
            }
            t1 = clock64();
            tc_commit(bar_done);
        }
        __syncwarp();
        const bool ok = mbar_wait_warp(bar_done, 0, env, DEV_TIMEOUT_MMA_FULL);
        if (lane == 0) {
            const long long t2 = clock64();
            const unsigned long long ns2 = globaltimer_ns();
            uint32_t smid;
            asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
            unsigned long long* o = p.out + 4 * (size_t)blockIdx.x;
            o[0] = (unsigned long long)(t1 - t0);
            o[1] = ok ? (unsigned long long)(t2 - t0) : 0ull;
            o[2] = ok ? ns2 - ns0 : 0ull;
            o[3] = smid;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace i8
