// C-ABI entry points of i8ops: argument validation, dispatch, tensor-map construction, launches.
// Everything that computes runs in the kernels included below; the host code only marshals.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <utility>

#include "../../include/i8ops.h"
#include "batched_tc.cuh"
#include "conv_slab.cuh"
#include "gemm_swap.cuh"
#include "gemm_tc.cuh"
#include "generic.cuh"
#include "mpc.cuh"
#include "probe.cuh"

namespace i8 {

// ------------------------------------------------------------------------------------------------ state
__device__ unsigned g_dev_status = 0;   // first bounded-wait expiry since the last query (0 = none)

constexpr int MAX_DEVICES = 64;

struct DeviceCtx {
    std::atomic<bool> ready{false};   // set last (release) by the one-time set-up; read without the lock afterwards
    int sm_count = 0;
    unsigned* dev_status = nullptr;   // device address of g_dev_status
    bool attr_set[32] = {};            // dynamic shared-memory opt-in done, per kernel instance
    void* ws = nullptr;               // workspace of the host-buffer variants
    size_t ws_bytes = 0;
    cudaStream_t s_in = nullptr, s_out = nullptr;   // copy streams of the host-buffer variants
    cudaEvent_t ev[2 * 8 + 2] = {};                 // chunk hand-over events (up to 8 row chunks)
    std::mutex host_mutex;                          // serialises the host-buffer variant: its calls share ws, s_in, s_out and ev
    std::atomic<bool> pool_ready{false};            // stream-ordered pool of the unfolded-convolution workspaces (made on first use)
    cudaMemPool_t pool = nullptr;
};

static DeviceCtx g_ctx[MAX_DEVICES];
static std::mutex g_mutex;
static int g_path_mode = 0;                      // 0 auto, 1 generic only, 2 two-SM tensor kernel whenever legal, 3 auto without the slab convolution
static uint64_t g_wait_limit_ns = 2000ull * 1000 * 1000;
static int g_pdl = 1;                            // programmatic dependent launch (I8OPS_PDL=0 turns it off)
static int g_tc2 = 1;                            // two-SM GEMM kernel for large shapes (I8OPS_TC2=0 turns it off)
static int g_conv_two_sm = -1;                   // CTA pairs for convolutions: -1 by rule, 0 never, 1 always (I8OPS_CONV2SM)
static int g_force_bn = -1;                      // tuning override from the environment (I8OPS_FORCE_BN)
static int g_tma_store = 1;                      // read-out of the wide tiles through TMA stores (I8OPS_TMA_STORE=0 turns it off)
static int g_sticky = 1;                         // column-sticky tile order for short-K problems (I8OPS_STICKY=0 turns it off)
static int g_tmap_cache = 1;                     // per-thread cache of encoded tensor maps (I8OPS_TMAP_CACHE=0 encodes every time)
static int g_swap = 1;                           // channel-major kernel: 0 never, 1 by rule, 2 wherever legal (I8OPS_SWAP)
static int g_swap_two_sm = -1;                   // channel-major kernel on CTA pairs: -1 by cost, 0 never, 1 whenever N > 128 (I8OPS_SWAP_2SM)
static int g_swap_stages = 0;                    // ring slots of the channel-major kernel: 0 = as many as fit (I8OPS_SWAP_STAGES)
static int g_swap_pw = 0;                        // strip width override for tuning (I8OPS_SWAP_PW)
static int g_slab = 1;                           // slab-resident stride-1 convolution kernel (I8OPS_SLAB=0 turns it off)
static int g_mpc_stream = 1;                     // streaming TinyMPC kernel: 0 off, 1 on, 2..4 ring slots (I8OPS_MPC_STREAM)
static int g_unfold = 1;                         // unfold + tensor GEMM for convolutions the im2col maps do not take (I8OPS_UNFOLD=0 turns it off)

static thread_local int t_last_path = I8_PATH_NONE;
static thread_local int t_last_cuda = 0;
static thread_local bool t_used_two_sm = false;
static thread_local bool t_used_swap = false;     // the last tensor-path launch was the channel-major kernel
static thread_local bool t_last_packed = false;   // the last GEMM ran on packed copies of its operands
static thread_local bool t_last_unfold = false;   // the last convolution ran as unfold + tensor GEMM
static thread_local bool t_tmap_failed = false;   // the last tensor-path attempt stopped at a tensor-map encoding (nothing launched)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode_tiled = nullptr;
typedef CUresult (*EncodeIm2colFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const int*, const int*, cuuint32_t, cuuint32_t, const cuuint32_t*,
                                   CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                   CUtensorMapFloatOOBfill);
static EncodeIm2colFn g_encode_im2col = nullptr;

static int tensor_path_used() {
    if (t_used_swap) return t_used_two_sm ? I8_PATH_CHANNEL_MAJOR_2SM : I8_PATH_CHANNEL_MAJOR;
    return t_used_two_sm ? I8_PATH_TENSOR_2SM : I8_PATH_TENSOR;
}

static int cuda_fail(cudaError_t e) {
    t_last_cuda = (int)e;
    return I8_ERR_CUDA;
}

#define CUDA_TRY(expr)                                   \
    do {                                                 \
        cudaError_t _e = (expr);                         \
        if (_e != cudaSuccess) return cuda_fail(_e);     \
    } while (0)

// Per-device set-up on first use: SM count, address of the status word, driver entry point.
static int get_ctx(DeviceCtx** out) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return cuda_fail(cudaErrorInvalidDevice);
    DeviceCtx& c = g_ctx[dev];
    if (c.ready.load(std::memory_order_acquire)) { *out = &c; return I8_OK; }   // the hot path takes no lock
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!c.ready.load(std::memory_order_relaxed)) {
        CUDA_TRY(cudaDeviceGetAttribute(&c.sm_count, cudaDevAttrMultiProcessorCount, dev));
        CUDA_TRY(cudaGetSymbolAddress((void**)&c.dev_status, g_dev_status));
        if (!g_encode_tiled) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult q;
            CUDA_TRY(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &q));
            if (q != cudaDriverEntryPointSuccess || !fn) return cuda_fail(cudaErrorNotSupported);
            g_encode_tiled = (EncodeTiledFn)fn;
            fn = nullptr;
            CUDA_TRY(cudaGetDriverEntryPointByVersion("cuTensorMapEncodeIm2col", &fn, 12000, cudaEnableDefault, &q));
            if (q != cudaDriverEntryPointSuccess || !fn) return cuda_fail(cudaErrorNotSupported);
            g_encode_im2col = (EncodeIm2colFn)fn;
        }
        const char* bn = getenv("I8OPS_FORCE_BN");
        if (bn) g_force_bn = atoi(bn);
        const char* c2 = getenv("I8OPS_CONV2SM");
        if (c2) g_conv_two_sm = atoi(c2);
        const char* tc2 = getenv("I8OPS_TC2");
        if (tc2) g_tc2 = atoi(tc2);
        const char* tst = getenv("I8OPS_TMA_STORE");
        if (tst) g_tma_store = atoi(tst);
        const char* sticky = getenv("I8OPS_STICKY");
        if (sticky) g_sticky = atoi(sticky);
        const char* slab = getenv("I8OPS_SLAB");
        if (slab) g_slab = atoi(slab);
        const char* mps = getenv("I8OPS_MPC_STREAM");
        if (mps) g_mpc_stream = atoi(mps);
        const char* unf = getenv("I8OPS_UNFOLD");
        if (unf) g_unfold = atoi(unf);
        const char* sw = getenv("I8OPS_SWAP");
        if (sw) g_swap = atoi(sw);
        const char* sw2 = getenv("I8OPS_SWAP_2SM");
        if (sw2) g_swap_two_sm = atoi(sw2);
        const char* sws = getenv("I8OPS_SWAP_STAGES");
        if (sws) g_swap_stages = atoi(sws);
        const char* swp = getenv("I8OPS_SWAP_PW");
        if (swp) g_swap_pw = atoi(swp);
        const char* tmc = getenv("I8OPS_TMAP_CACHE");
        if (tmc) g_tmap_cache = atoi(tmc);
        const char* pdl = getenv("I8OPS_PDL");
        if (pdl) g_pdl = atoi(pdl);
        c.ready.store(true, std::memory_order_release);
    }
    *out = &c;
    return I8_OK;
}

// ------------------------------------------------------------------------------------------------ tensor maps
// Encoding a tensor map is a driver call of about a microsecond, and a call needs two or three of them, which is as
// much as a small problem's kernel time.  Maps depend only on the base address and the geometry, so each host thread
// keeps the ones it encoded in a small direct-mapped cache (no lock: the cache is thread-local) keyed on everything
// that goes into the encoding, the base pointer included.
struct TmapKey {
    uint64_t base;
    uint64_t dims[5];
    uint64_t strides[4];
    uint32_t box[5];
    uint32_t rank, swizzle, kind;     // kind: 0 tiled, 1 im2col
    int32_t lower[2], upper[2];       // im2col: bounding-box corners
    uint32_t estr[5];                 // traversal strides
    uint32_t channels, pixels;        // im2col: channels per pixel, pixels per column
};
struct TmapEntry {
    TmapKey key;
    alignas(64) CUtensorMap map;
    bool valid;
};
constexpr int TMAP_CACHE_SETS = 32, TMAP_CACHE_WAYS = 4;      // four ways: the two or three maps of one call never evict each other
static thread_local TmapEntry t_tmap_cache[TMAP_CACHE_SETS][TMAP_CACHE_WAYS];
static thread_local uint8_t t_tmap_next[TMAP_CACHE_SETS];     // way to replace next, per set
static thread_local uint64_t t_tmap_hits = 0, t_tmap_misses = 0;

static uint32_t tmap_hash(const TmapKey& k) {
    const uint32_t* w = reinterpret_cast<const uint32_t*>(&k);
    uint32_t h = 2166136261u;
    for (size_t i = 0; i < sizeof(TmapKey) / 4; i++) h = (h ^ w[i]) * 16777619u;
    return h ^ (h >> 15);
}

static int encode_tmap(CUtensorMap* tm, const TmapKey& k) {
    cuuint64_t gdim[5], gstr[4];
    cuuint32_t bx[5], es[5];
    for (uint32_t i = 0; i < k.rank; i++) { gdim[i] = k.dims[i]; bx[i] = k.box[i]; es[i] = k.estr[i]; }
    for (uint32_t i = 0; i + 1 < k.rank; i++) gstr[i] = k.strides[i];
    CUresult r;
    if (k.kind == 0)
        r = g_encode_tiled(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, k.rank, reinterpret_cast<void*>(k.base), gdim, gstr, bx, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, (CUtensorMapSwizzle)k.swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    else
        r = g_encode_im2col(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, k.rank, reinterpret_cast<void*>(k.base), gdim, gstr, k.lower, k.upper,
                            k.channels, k.pixels, es, CU_TENSOR_MAP_INTERLEAVE_NONE, (CUtensorMapSwizzle)k.swizzle,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { t_last_cuda = (int)cudaErrorInvalidValue; t_tmap_failed = true; return I8_ERR_CUDA; }
    return I8_OK;
}

static int cached_tmap(CUtensorMap* tm, const TmapKey& k) {
    if (!g_tmap_cache) return encode_tmap(tm, k);
    const uint32_t set = tmap_hash(k) % TMAP_CACHE_SETS;
    for (int w = 0; w < TMAP_CACHE_WAYS; w++) {
        const TmapEntry& e = t_tmap_cache[set][w];
        if (e.valid && memcmp(&e.key, &k, sizeof(TmapKey)) == 0) {
            *tm = e.map;
            t_tmap_hits++;
            return I8_OK;
        }
    }
    t_tmap_misses++;
    int rc = encode_tmap(tm, k);
    if (rc) return rc;
    TmapEntry& e = t_tmap_cache[set][t_tmap_next[set]];
    t_tmap_next[set] = (uint8_t)((t_tmap_next[set] + 1) % TMAP_CACHE_WAYS);
    e.key = k; e.map = *tm; e.valid = true;
    return I8_OK;
}

// Tiled byte tensor of rank 2..5, innermost dimension contiguous, zero fill outside.
static int make_tmap(CUtensorMap* tm, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                     const uint32_t* box, CUtensorMapSwizzle swz) {
    TmapKey k;
    memset(&k, 0, sizeof(k));
    k.base = reinterpret_cast<uint64_t>(base);
    k.rank = (uint32_t)rank; k.swizzle = (uint32_t)swz; k.kind = 0;
    for (int i = 0; i < rank; i++) { k.dims[i] = dims[i]; k.box[i] = box[i]; k.estr[i] = 1; }
    for (int i = 0; i + 1 < rank; i++) k.strides[i] = strides_bytes[i];
    return cached_tmap(tm, k);
}

// im2col-mode map over dense NHWC activations: `channels` bytes x `pixels` output positions per load.
static int make_tmap_im2col(CUtensorMap* tm, const void* x, int N, int H, int W, int C, int R, int S, int stride_h, int stride_w,
                            int pad_h, int pad_w, int channels, int pixels, CUtensorMapSwizzle swz) {
    TmapKey k;
    memset(&k, 0, sizeof(k));
    k.base = reinterpret_cast<uint64_t>(x);
    k.rank = 4; k.swizzle = (uint32_t)swz; k.kind = 1;
    k.dims[0] = (uint64_t)C; k.dims[1] = (uint64_t)W; k.dims[2] = (uint64_t)H; k.dims[3] = (uint64_t)N;
    k.strides[0] = (uint64_t)C; k.strides[1] = (uint64_t)W * C; k.strides[2] = (uint64_t)H * W * C;
    k.lower[0] = -pad_w; k.lower[1] = -pad_h;
    k.upper[0] = pad_w - (S - 1); k.upper[1] = pad_h - (R - 1);
    k.estr[0] = 1; k.estr[1] = (uint32_t)stride_w; k.estr[2] = (uint32_t)stride_h; k.estr[3] = 1;
    k.channels = (uint32_t)channels; k.pixels = (uint32_t)pixels;
    return cached_tmap(tm, k);
}

// Launch on `st`; with programmatic stream serialisation the kernel may be scheduled while its predecessor in
// the stream drains (the kernels wait for their dependencies before touching global memory).
template <typename... KArgs, typename... Args>
static cudaError_t launch_kernel(void (*kern)(KArgs...), bool overlap, int cluster, int grid, int block, size_t smem,
                                 cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (g_pdl && overlap) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        n++;
    }
    if (cluster > 1) {                      // CTA pairs: clusters of `cluster` consecutive CTAs
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cluster;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        n++;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ------------------------------------------------------------------------------------------------ launches
static CUtensorMapSwizzle swizzle_for(int cb) {
    return cb == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (cb == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
}

template <int BN, int STAGES, bool CONV, int EPI_WARPS, int NPROD, bool TWO_SM>
static int launch_tc(DeviceCtx* ctx, int slot, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC,
                     GemmTcParams& p, cudaStream_t st) {
    using L = TcSmem<BN, STAGES, TWO_SM>;
    auto kern = gemm_i8_tc_kernel<BN, STAGES, CONV, EPI_WARPS, NPROD, TWO_SM>;
    if (!ctx->attr_set[slot]) {
        CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::DYN_BYTES));
        ctx->attr_set[slot] = true;
    }
    const int workers = TWO_SM ? ctx->sm_count / 2 : ctx->sm_count;          // CTAs, or CTA pairs
    const int used = p.sched.num_tiles < workers ? p.sched.num_tiles : workers;
    // short kernels gain from overlapping their launch with the predecessor's tail; long ones do not need it
    const bool overlap = !TWO_SM && 2.0 * p.M * p.N * p.K < 4e10;
    CUDA_TRY(launch_kernel(kern, overlap, TWO_SM ? 2 : 1, TWO_SM ? 2 * used : used, 32 * (1 + NPROD) + 32 * EPI_WARPS, L::DYN_BYTES,
                           st, tmA, tmB, tmC, p));
    return I8_OK;
}

// ------------------------------------------------------------------------------------------------ planning
// Shape classes of the paper's schedule-reuse experiment: a schedule found for one shape is reused for shapes of the
// same aspect class (square, column-dominant = tall and narrow, row-dominant = short and wide).
static int shape_class(int M, int N) {
    if ((int64_t)M >= 8 * (int64_t)N) return 1;
    if ((int64_t)N >= 8 * (int64_t)M) return 2;
    return 0;
}

// One recorded schedule per class: the choices the planner would otherwise take from its cost model.  An entry with a
// base shape applies to shapes whose M, N and K each lie within a factor of four of the base's (the "nearby shapes" of
// the paper's reuse table); an entry without one (base_m == 0) applies to the whole class.
struct ClassPlan {
    int valid;
    int base_m, base_n, base_k;
    int tile_n;          // 64, 128, 256; 0 = cost model
    int cta_group;       // 1, 2; 0 = crossover rule
    int raster_group;    // block rows per raster group; 0 = default
    int sticky;          // 1 = column-sticky order where legal, 0 = never, -1 = rule
};
// Seeds: the tuned plans of the two workload configurations with a clear class (8192^3 on CTA pairs with 16-row raster
// groups; the 262144 x 64 x 256 stream on 64-wide tiles with B resident).
static ClassPlan g_class_plan[3] = {
    {1, 8192, 8192, 8192, 256, 2, 16, -1},
    {1, 262144, 64, 256, 64, 1, 16, -1},
    {0, 0, 0, 0, 0, 0, 0, -1},
};

static bool near_base(int v, int base) { return (int64_t)v * 4 >= base && (int64_t)v <= (int64_t)base * 4; }

static const ClassPlan* recorded_plan(int M, int N, int K) {
    const ClassPlan& e = g_class_plan[shape_class(M, N)];
    if (!e.valid) return nullptr;
    if (e.base_m && !(near_base(M, e.base_m) && near_base(N, e.base_n) && near_base(K, e.base_k))) return nullptr;
    return &e;
}

// Tile width.  Cost model in SM cycles: every wave of tiles pays, per 128-byte K block, an operand-delivery
// bound of 256 + 2*BN, plus a fixed 400 per tile; the last tile's read-out (about 14 cycles per column) is
// exposed.  The width with the lowest total wins; ties go to the wider tile.
static int choose_bn(int M, int N, int num_kb, int sm_count, const ClassPlan* rec) {
    if (g_force_bn == 64 || g_force_bn == 128 || g_force_bn == 256) return g_force_bn;
    const int recorded = rec ? rec->tile_n : 0;
    if (recorded && (recorded == 64 || recorded - 64 < ((N + 63) / 64) * 64)) return recorded;
    const int cands[3] = {256, 128, 64};
    int best = 64;
    double best_cost = 1e300;
    const int m_tiles = (M + BM - 1) / BM;
    for (int i = 0; i < 3; i++) {
        const int bn = cands[i];
        if (bn > 64 && bn - 64 >= ((N + 63) / 64) * 64) continue;   // tile mostly empty
        const int64_t tiles = (int64_t)m_tiles * ((N + bn - 1) / bn);
        const int64_t waves = (tiles + sm_count - 1) / sm_count;
        const double cost = (double)waves * ((double)num_kb * (256.0 + 2.0 * bn) + 400.0) + 14.0 * bn;
        if (cost < best_cost - 1e-9) { best_cost = cost; best = bn; }
    }
    return best;
}

// Everything the host decides about one launch of the large-tile kernel.  The launch code and the plan query both get
// it from plan_tc(), so the query reports what runs.
struct TcPlan {
    int two_sm, bn, stages, tile_m;
    int workers;                 // CTAs (one-SM) or CTA pairs launched
    int m_tiles, n_tiles, num_tiles;
    int group_m, sticky, col_base, col_rem;
    int b_resident;
    int shape_cls;
};
static thread_local i8_plan t_last_plan = {};     // what the last launch of a tensor kernel by this thread used
static void fill_plan(const TcPlan& pl, i8_plan* out);

// CTA pairs: their larger tiles and cluster set-up cost about 1.5 us more per launch, which pays once there is at least
// one full wave of 256-row tiles and enough K per cluster (measured crossover: waves x K blocks ~ 48).
static bool pair_pays(int M, int N, int bn, int num_kb, int sm_count) {
    const int clusters = sm_count / 2;
    const int64_t tiles2 = (int64_t)((M + 255) / 256) * ((N + bn - 1) / bn);
    const int64_t waves2 = (tiles2 + clusters - 1) / clusters;
    return tiles2 >= clusters && waves2 * num_kb >= 48;
}

// conv: the operand A comes through im2col loads (three two-SM instances exist); GEMM: the two-SM instance is 256 wide.
// num_kb = 128-byte K blocks, num_iters = ring slots per tile, cb = bytes of K per sub-block.
static TcPlan plan_tc(bool conv, int M, int N, int K, int num_kb, int num_iters, int num_kblocks, int cb, int sm_count) {
    TcPlan pl = {};
    pl.shape_cls = shape_class(M, N);
    const ClassPlan* rec = conv ? nullptr : recorded_plan(M, N, K);
    bool two_sm;
    int bn;
    if (conv) {
        bn = choose_bn(M, N, num_kb, sm_count, nullptr);
        two_sm = g_path_mode == 2 || g_conv_two_sm == 1;
        if (g_tc2 && g_conv_two_sm != 0 && g_force_bn < 0 && pair_pays(M, N, bn, num_kb, sm_count)) two_sm = true;
    } else {
        bool want2 = g_tc2 && pair_pays(M, N, 256, num_kb, sm_count);
        if (rec && rec->cta_group == 1) want2 = false;
        if (rec && rec->cta_group == 2 && g_tc2) want2 = true;
        two_sm = g_force_bn < 0 && (want2 || g_path_mode == 2);
        bn = two_sm ? 256 : choose_bn(M, N, num_kb, sm_count, rec);
    }
    pl.two_sm = two_sm ? 1 : 0;
    pl.bn = bn;
    pl.tile_m = two_sm ? 2 * BM : BM;
    // ring slots per instance (must match the launch table in run_tc)
    // (64-wide GEMM tiles: 6 slots measured 4 % faster than 8 on the tall-skinny stream, as deep rings also were on the batched kernel)
    pl.stages = two_sm ? (bn == 256 ? 6 : 8) : (bn == 256 ? 4 : (bn == 128 ? 6 : (conv ? 8 : 6)));
    pl.m_tiles = (M + pl.tile_m - 1) / pl.tile_m;
    pl.n_tiles = (N + bn - 1) / bn;
    pl.num_tiles = pl.m_tiles * pl.n_tiles;
    const int max_workers = two_sm ? sm_count / 2 : sm_count;
    pl.workers = pl.num_tiles < max_workers ? pl.num_tiles : max_workers;
    pl.group_m = (rec && rec->raster_group > 0) ? rec->raster_group : 16;   // 16: measured best of 2..32 on 8192^3 for the two-SM kernel
    // Column-sticky order for short-K problems with several tiles per worker: rebuilding the epilogue constants for
    // a new block column costs about as much as a short tile, so a worker keeps its column if that needs no more
    // rounds than the raster order.
    pl.sticky = 0; pl.col_base = 0; pl.col_rem = 0;
    {
        const int nt = pl.n_tiles, mt = pl.m_tiles, workers = max_workers;
        const int pref = rec ? rec->sticky : -1;
        const bool legal = nt > 1 && workers >= 2 * nt && pl.num_tiles > workers;
        if (g_sticky && legal && pref != 0 && (pref == 1 || num_iters <= 16)) {
            const int base = workers / nt;
            const int rounds_sticky = (mt + base - 1) / base;
            const int rounds_raster = (pl.num_tiles + workers - 1) / workers;
            if (pref == 1 || rounds_sticky <= rounds_raster) { pl.sticky = 1; pl.col_base = base; pl.col_rem = workers % nt; }
        }
    }
    // resident B: one block column, and all of B's K blocks fit the ring's B region
    const int b_rows = two_sm ? bn / 2 : bn;
    pl.b_resident = (pl.n_tiles == 1 && (int64_t)num_kblocks * b_rows * cb <= (int64_t)pl.stages * b_rows * BK) ? 1 : 0;
    return pl;
}

// Common tail of the tensor paths: B's tensor map (an N x K matrix with K contiguous), the tile schedule,
// and the launch of the instance that matches the tile width.
struct RawOut { int32_t* D = nullptr; int64_t ldd = 0; int accumulate = 0; };
// Independent problems of one shape in one launch: problem b starts a_rpp / b_rpp / c_rpp rows further in the stacked
// 2-D views of A / B / C, its bias bias_bs entries further; mt = block rows per problem.
struct BatchInfo { int batch = 1, mt = 0; int64_t a_rpp = 0, b_rpp = 0, c_rpp = 0, bias_bs = 0; };

static int run_tc(DeviceCtx* ctx, bool conv, const TcPlan& pl, const CUtensorMap& tmA, const KLoop& kl, const int8_t* B,
                  int64_t ldb, int8_t* C, int64_t ldc, const int32_t* bias, const int32_t* mult, const int32_t* shift,
                  int per_channel, int M, int N, int K, int relu, cudaStream_t st, const RawOut& raw = RawOut(),
                  const BatchInfo& bt = BatchInfo()) {
    const bool two_sm = pl.two_sm != 0;
    const int bn = pl.bn;
    const int b_rows = two_sm ? bn / 2 : bn;           // rows of the B tile one CTA loads
    fill_plan(pl, &t_last_plan);
    t_used_two_sm = two_sm;
    CUtensorMap tmB;
    if (kl.b_mn) {
        // B stored with N contiguous: K rows of 128 (64-wide tiles: 64) bytes of N
        const uint32_t mnw = b_rows >= 128 ? 128u : 64u;
        const uint64_t dims[2] = {(uint64_t)N, (uint64_t)((bt.batch - 1) * bt.b_rpp + K)};
        const uint64_t str[1] = {(uint64_t)ldb};
        const uint32_t box[2] = {mnw, (uint32_t)BK};
        int rc = make_tmap(&tmB, B, 2, dims, str, box, mnw == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B);
        if (rc) return rc;
    } else {
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)((bt.batch - 1) * bt.b_rpp + N)};
        const uint64_t str[1] = {(uint64_t)ldb};
        const uint32_t box[2] = {(uint32_t)kl.cb, (uint32_t)b_rows};
        int rc = make_tmap(&tmB, B, 2, dims, str, box, swizzle_for(kl.cb));
        if (rc) return rc;
    }
    GemmTcParams p;
    p.batch_mt = bt.batch > 1 ? bt.mt : 0;
    p.inv_bmt = bt.mt <= 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)bt.mt);
    p.a_rpp = (int)bt.a_rpp; p.b_rpp = (int)bt.b_rpp; p.c_rpp = bt.c_rpp; p.bias_bs = bt.batch > 1 ? bt.bias_bs : 0;
    p.C = C; p.ldc = ldc; p.bias = bias; p.mult = mult; p.shift = shift;
    p.per_channel = per_channel; p.relu = relu; p.M = M; p.N = N; p.K = K;
    p.c_vec_ok = raw.D ? (aligned16(raw.D) && raw.ldd % 4 == 0) : (aligned16(C) && (ldc % 16 == 0));
    p.D = raw.D; p.ldd = raw.ldd; p.raw = raw.D ? 1 : 0; p.accumulate = raw.accumulate;
    // wide tiles hand their int8 output to the TMA engine as 32-row x 64-byte boxes; needs a 16-byte aligned C and an N
    // that is a multiple of 16: the copy engine clips a box at the tensor's edge in 16-byte units, so with a ragged N
    // it would write up to 15 bytes past the last column
    CUtensorMap tmC = tmB;
    p.tma_store = 0;
    if (g_tma_store && !raw.D && bn >= 128 && p.c_vec_ok && N % 16 == 0 && bt.batch == 1) {
        const uint64_t dims[2] = {(uint64_t)N, (uint64_t)M};
        const uint64_t str[1] = {(uint64_t)ldc};
        const uint32_t box[2] = {64, 32};
        int rc = make_tmap(&tmC, C, 2, dims, str, box, CU_TENSOR_MAP_SWIZZLE_64B);
        if (rc) return rc;
        p.tma_store = 1;
    }
    p.sched.m_tiles = pl.m_tiles;
    p.sched.n_tiles = pl.n_tiles;
    p.sched.num_tiles = pl.num_tiles;
    p.sched.group_m = pl.group_m;
    p.sched.sticky = pl.sticky; p.sched.col_base = pl.col_base; p.sched.col_rem = pl.col_rem;
    {
        auto inv32 = [](int d) { return d <= 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)d); };
        p.sched.inv_nt = inv32(p.sched.n_tiles);
        p.sched.inv_width = inv32(p.sched.group_m * p.sched.n_tiles);
        p.sched.inv_gm = inv32(p.sched.group_m);
        p.sched.inv_step = inv32(pl.workers);
        const int last = p.sched.m_tiles % p.sched.group_m;
        p.sched.inv_last = inv32(last ? last : p.sched.group_m);
        p.sched.inv_cb = pl.sticky ? inv32(pl.col_base) : 0xffffffffu;
        p.sched.inv_cb1 = pl.sticky ? inv32(pl.col_base + 1) : 0xffffffffu;
    }
    p.kl = kl;
    p.kl.b_resident = kl.b_mn ? 0 : pl.b_resident;            // the resident-B fetch is written for K-major B only
    p.wait_limit_cycles = (long long)(g_wait_limit_ns * 2);   // SM clock stays below 2 GHz: at least the asked time
    p.dev_status = ctx->dev_status;
    if (two_sm) {
        if (conv) {
            switch (bn) {
                case 256: return launch_tc<256, 6, true, 8, 2, true>(ctx, 8, tmA, tmB, tmC, p, st);
                case 128: return launch_tc<128, 8, true, 8, 2, true>(ctx, 9, tmA, tmB, tmC, p, st);
                default:  return launch_tc<64, 8, true, 8, 2, true>(ctx, 10, tmA, tmB, tmC, p, st);
            }
        }
        return launch_tc<256, 6, false, 8, 1, true>(ctx, 7, tmA, tmB, tmC, p, st);
    }
    if (conv) {
        switch (bn) {
            case 256: return launch_tc<256, 4, true, 8, 2, false>(ctx, 3, tmA, tmB, tmC, p, st);
            case 128: return launch_tc<128, 6, true, 8, 2, false>(ctx, 4, tmA, tmB, tmC, p, st);
            default:  return launch_tc<64, 8, true, 8, 2, false>(ctx, 5, tmA, tmB, tmC, p, st);
        }
    }
    switch (bn) {
        case 256: return launch_tc<256, 4, false, 8, 1, false>(ctx, 0, tmA, tmB, tmC, p, st);
        case 128: return launch_tc<128, 6, false, 8, 1, false>(ctx, 1, tmA, tmB, tmC, p, st);
        default:  return launch_tc<64, 6, false, 8, 1, false>(ctx, 2, tmA, tmB, tmC, p, st);
    }
}

static int run_gemm_swap(DeviceCtx* ctx, const int8_t* A, int64_t lda, const int8_t* B, int64_t ldb, int8_t* C, int64_t ldc,
                         const int32_t* bias, const int32_t* mult, const int32_t* shift, int per_channel, int M, int N, int K,
                         int relu, cudaStream_t st, const float* fscale = nullptr);
static bool swap_wanted(bool conv, int M, int N, int K, int num_kb, int num_iters, int num_kblocks, int cb, int sm_count);

static KLoop gemm_kloop(int K) {
    KLoop kl{};
    kl.cb = BK; kl.nsub = 1; kl.num_kblocks = (K + BK - 1) / BK;
    kl.num_iters = kl.num_kblocks;
    kl.mmas_last = ((K - (kl.num_iters - 1) * BK) + 31) / 32;
    return kl;
}

// a_mn / b_mn: the operand is stored with M (A) or N (B) contiguous instead of K; lda / ldb is then the stride between K rows.
static int run_gemm_tc(DeviceCtx* ctx, const int8_t* A, int64_t lda, const int8_t* B, int64_t ldb, int8_t* C, int64_t ldc,
                       const int32_t* bias, const int32_t* mult, const int32_t* shift, int per_channel, int M, int N,
                       int K, int relu, cudaStream_t st, const RawOut& raw = RawOut(), int a_mn = 0, int b_mn = 0) {
    KLoop kl = gemm_kloop(K);
    kl.a_mn = a_mn; kl.b_mn = b_mn;
    t_used_swap = false;
    if (!raw.D && !a_mn && !b_mn && swap_wanted(false, M, N, K, kl.num_kblocks, kl.num_iters, kl.num_kblocks, BK, ctx->sm_count)) {
        int rc = run_gemm_swap(ctx, A, lda, B, ldb, C, ldc, bias, mult, shift, per_channel, M, N, K, relu, st);
        if (rc != I8_ERR_UNSUPPORTED) { t_used_swap = rc == I8_OK; return rc; }
    }
    const TcPlan pl = plan_tc(false, M, N, K, kl.num_kblocks, kl.num_iters, kl.num_kblocks, BK, ctx->sm_count);
    CUtensorMap tmA;
    const uint64_t dims_k[2] = {(uint64_t)K, (uint64_t)M}, dims_m[2] = {(uint64_t)M, (uint64_t)K};
    const uint64_t str[1] = {(uint64_t)lda};
    const uint32_t box[2] = {BK, BM};                  // K-major: 128 bytes of K x 128 rows; MN-major: 128 rows x 128 of K
    int rc = make_tmap(&tmA, A, 2, a_mn ? dims_m : dims_k, str, box, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    return run_tc(ctx, false, pl, tmA, kl, B, ldb, C, ldc, bias, mult, shift, per_channel, M, N, K, relu, st, raw);
}

// A batch of equal-shape problems (K-contiguous operands, batch strides that are whole numbers of rows) as ONE launch of
// the large-tile kernel on single CTAs: the tile schedule runs over the block rows of all problems.
static int run_gemm_tc_batched(DeviceCtx* ctx, const int8_t* A, int64_t lda, int64_t a_bs, const int8_t* B, int64_t ldb, int64_t b_bs,
                               int8_t* C, int64_t ldc, int64_t c_bs, const int32_t* bias, int64_t bias_bs, const int32_t* mult,
                               const int32_t* shift, int per_channel, int batch, int M, int N, int K, int relu, cudaStream_t st,
                               int b_mn) {
    if (a_bs % lda || b_bs % ldb || c_bs % ldc) return I8_ERR_UNSUPPORTED;
    BatchInfo bt;
    bt.batch = batch; bt.a_rpp = a_bs / lda; bt.b_rpp = b_bs / ldb; bt.c_rpp = c_bs / ldc; bt.bias_bs = bias_bs;
    bt.mt = (M + BM - 1) / BM;
    const int64_t rows_a = (batch - 1) * bt.a_rpp + M, rows_b = (batch - 1) * bt.b_rpp + (b_mn ? K : N);
    if (rows_a >= (1ll << 31) - BM || rows_b >= (1ll << 31) - 256 || (int64_t)bt.mt * batch >= (1ll << 24)) return I8_ERR_UNSUPPORTED;
    KLoop kl = gemm_kloop(K);
    kl.b_mn = b_mn;
    TcPlan pl = {};
    pl.shape_cls = shape_class(M, N);
    pl.two_sm = 0;
    pl.bn = choose_bn((int)((int64_t)bt.mt * batch > 65536 ? 65536 * BM : bt.mt * batch * BM), N, kl.num_kblocks, ctx->sm_count, nullptr);
    pl.tile_m = BM;
    pl.stages = pl.bn == 256 ? 4 : 6;
    pl.m_tiles = bt.mt * batch;
    pl.n_tiles = (N + pl.bn - 1) / pl.bn;
    if ((int64_t)pl.m_tiles * pl.n_tiles >= (1ll << 30)) return I8_ERR_UNSUPPORTED;
    pl.num_tiles = pl.m_tiles * pl.n_tiles;
    pl.workers = pl.num_tiles < ctx->sm_count ? pl.num_tiles : ctx->sm_count;
    pl.group_m = 16;
    pl.sticky = 0; pl.col_base = 0; pl.col_rem = 0; pl.b_resident = 0;
    CUtensorMap tmA;
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)rows_a};
    const uint64_t str[1] = {(uint64_t)lda};
    const uint32_t box[2] = {BK, BM};
    int rc = make_tmap(&tmA, A, 2, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    return run_tc(ctx, false, pl, tmA, kl, B, ldb, C, ldc, bias, mult, shift, per_channel, M, N, K, relu, st, RawOut(), bt);
}

// ------------------------------------------------------------------------------------------------ channel-major kernel
// Plan of one launch of gemm_i8_swap_kernel: strip width, ring depth, shared-memory layout.
struct SwapPlan {
    int two_sm, pw, b_rows, stages, workers, m_tiles, n_blocks, num_tiles, tmem_cols;
    int off_b, off_bar, smem_bytes;
    double cycles;             // the cost model's estimate for the whole launch
};
static void fill_plan_swap(const SwapPlan& sp, int M, int N, i8_plan* out) {
    out->shape_class = shape_class(M, N);
    out->kernel = 1;
    out->tile_m = sp.pw;                        // rows of C per tile: the strip
    out->tile_n = sp.two_sm ? 256 : 128;        // columns of C per tile: the channel block
    out->stages = sp.stages;
    out->cta_group = sp.two_sm ? 2 : 1;
    out->raster_group = 0;
    out->sticky = 0;
    out->m_tiles = sp.m_tiles;
    out->n_tiles = sp.n_blocks;
    out->workers = sp.workers;
    out->waves = sp.workers ? (sp.num_tiles + sp.workers - 1) / sp.workers : 0;
    out->b_resident = 0;
    out->epilogue_warps = SWAP_EPI_WARPS;
}

static void fill_plan(const TcPlan& pl, i8_plan* out) {
    out->shape_class = pl.shape_cls;
    out->kernel = 0;
    out->tile_m = pl.tile_m;
    out->tile_n = pl.bn;
    out->stages = pl.stages;
    out->cta_group = pl.two_sm ? 2 : 1;
    out->raster_group = pl.group_m;
    out->sticky = pl.sticky;
    out->m_tiles = pl.m_tiles;
    out->n_tiles = pl.n_tiles;
    out->workers = pl.workers;
    out->waves = pl.workers ? (pl.num_tiles + pl.workers - 1) / pl.workers : 0;
    out->b_resident = pl.b_resident;
    out->epilogue_warps = 8;
}


// Strip width: every candidate (multiples of 16) is priced as waves x (ring slots per tile x cycles per slot + a fixed
// cost per tile) + the exposed read-out of the last tile.  A slot's cycles are the larger of its four instructions
// (pw / 2 cycles each, at least 48: narrower instructions are bound by operand reads) and its operand bytes at the
// ~80 bytes per clock an SM draws from L2.
static SwapPlan plan_swap(int M, int N, int num_iters, bool two_sm, int sm_count) {
    SwapPlan best = {};
    best.cycles = 1e300;
    const int tile_ch = two_sm ? 256 : 128;
    const int n_blocks = (N + tile_ch - 1) / tile_ch;
    const int max_workers = two_sm ? sm_count / 2 : sm_count;
    for (int pw = 256; pw >= 16; pw -= 16) {
        if (g_swap_pw && pw != g_swap_pw) continue;
        const int m_tiles = (M + pw - 1) / pw;
        const int64_t tiles = (int64_t)m_tiles * n_blocks;
        if (tiles >= (1ll << 30)) continue;
        const int64_t waves = (tiles + max_workers - 1) / max_workers;
        const int b_rows = two_sm ? pw / 2 : pw;
        const double mma = 4.0 * (pw / 2 > 48 ? pw / 2 : 48);
        const double feed = (16384.0 + 128.0 * b_rows) / 80.0;
        const double cyc = (double)waves * ((double)num_iters * (mma > feed ? mma : feed) + 500.0) + 4.0 * pw;
        if (cyc < best.cycles - 1e-9) {
            best.cycles = cyc; best.pw = pw; best.b_rows = b_rows; best.m_tiles = m_tiles; best.n_blocks = n_blocks;
            best.num_tiles = (int)tiles; best.workers = (int)(tiles < max_workers ? tiles : max_workers);
        }
    }
    best.two_sm = two_sm ? 1 : 0;
    if (!best.pw) return best;
    int cols = 32;
    while (cols < 2 * best.pw) cols *= 2;
    best.tmem_cols = cols;
    const int b_stage = best.b_rows * 128;
    const int stage_bytes = 16384 + b_stage;
    const int fixed = (2 * SWAP_MAX_STAGES + 4) * 8 + 16;
    int stages = (226 * 1024 - fixed) / stage_bytes;
    if (stages > SWAP_MAX_STAGES) stages = SWAP_MAX_STAGES;
    if (g_swap_stages >= 2 && g_swap_stages < stages) stages = g_swap_stages;
    best.stages = stages;
    best.off_b = stages * 16384;
    best.off_bar = best.off_b + stages * b_stage;
    best.smem_bytes = best.off_bar + fixed + 1024;
    return best;
}

// CTA pairs halve the activation bytes each CTA pulls from L2 but cost a fixed amount per launch (cluster scheduling,
// two cluster barriers, the paired commit): on the 12544 x 256 x 1152 / 2304 convolutions the model's 1270- / 2540-cycle
// advantage for pairs is a 0.63 / 0.55 us loss in fact (8.37 -> 7.72 and 10.2 -> 9.65 us on single CTAs), i.e. 2300-3500
// cycles.  Pairs are taken only where the model still sees them ahead by more than that.
static const double SWAP_PAIR_FIXED_CYCLES = 4000.0;
static SwapPlan plan_swap_auto(int M, int N, int num_iters, int sm_count) {
    const SwapPlan one = plan_swap(M, N, num_iters, false, sm_count);
    if (N <= 128 || g_swap_two_sm == 0 || g_path_mode == 6) return one;
    const SwapPlan two = plan_swap(M, N, num_iters, true, sm_count);
    if (g_swap_two_sm == 1 || g_path_mode == 5 || !one.pw) return two;
    return two.pw && two.cycles + SWAP_PAIR_FIXED_CYCLES < one.cycles ? two : one;
}

template <bool CONV, bool TWO_SM>
static int launch_swap(DeviceCtx* ctx, int slot, const SwapPlan& pl, const CUtensorMap& tmW, const CUtensorMap& tmX, const SwapParams& p,
                       cudaStream_t st) {
    auto kern = gemm_i8_swap_kernel<CONV, TWO_SM>;
    if (!ctx->attr_set[slot]) {
        CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        ctx->attr_set[slot] = true;
    }
    CUDA_TRY(launch_kernel(kern, true, TWO_SM ? 2 : 1, TWO_SM ? 2 * pl.workers : pl.workers, 32 * (CONV ? 3 : 2) + 32 * SWAP_EPI_WARPS,
                           (size_t)pl.smem_bytes, st, tmW, tmX, p));
    return I8_OK;
}

// W: [N][ldw] K-contiguous weights (the caller's B); tmX: the map of the other operand, built by the caller for the
// plan's b_rows.  C row-major [M][ldc].
static int run_swap(DeviceCtx* ctx, bool conv, const SwapPlan& pl, const CUtensorMap& tmX, const KLoop& kl, const int8_t* W, int64_t ldw,
                    int8_t* C, int64_t ldc, const int32_t* bias, const int32_t* mult, const int32_t* shift, int per_channel,
                    int M, int N, int K, int relu, cudaStream_t st, const float* fscale = nullptr) {
    CUtensorMap tmW;
    {
        const uint64_t dims[2] = {(uint64_t)K, (uint64_t)N};
        const uint64_t str[1] = {(uint64_t)ldw};
        const uint32_t box[2] = {(uint32_t)kl.cb, (uint32_t)BM};
        int rc = make_tmap(&tmW, W, 2, dims, str, box, swizzle_for(kl.cb));
        if (rc) return rc;
    }
    SwapParams p;
    p.C = C; p.ldc = ldc; p.bias = bias; p.mult = mult; p.shift = shift; p.per_channel = per_channel; p.relu = relu;
    p.fscale = fscale;
    p.M = M; p.N = N; p.K = K;
    p.pw = pl.pw; p.b_rows = pl.b_rows;
    p.c_word_ok = ((reinterpret_cast<uintptr_t>(C) & 3u) == 0 && ldc % 4 == 0 && N % 4 == 0) ? 1 : 0;
    p.m_tiles = pl.m_tiles; p.n_blocks = pl.n_blocks; p.num_tiles = pl.num_tiles;
    p.inv_nb = pl.n_blocks <= 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)pl.n_blocks);
    p.stages = pl.stages; p.b_stage_bytes = pl.b_rows * 128; p.tmem_cols = pl.tmem_cols;
    p.off_b = pl.off_b; p.off_bar = pl.off_bar;
    p.kl = kl;
    p.kl.b_resident = 0;
    p.wait_limit_cycles = (long long)(g_wait_limit_ns * 2);
    p.dev_status = ctx->dev_status;
    t_used_two_sm = pl.two_sm != 0;
    fill_plan_swap(pl, M, N, &t_last_plan);
    if (conv) return pl.two_sm ? launch_swap<true, true>(ctx, 21, pl, tmW, tmX, p, st) : launch_swap<true, false>(ctx, 22, pl, tmW, tmX, p, st);
    return pl.two_sm ? launch_swap<false, true>(ctx, 23, pl, tmW, tmX, p, st) : launch_swap<false, false>(ctx, 24, pl, tmW, tmX, p, st);
}

// Whether a problem goes to the channel-major kernel.  Forced (path mode 4, I8OPS_SWAP=2): whenever it is legal.  By
// rule: its read-out costs more per output than the large-tile kernel's (a transpose in registers), so it is taken only
// where its freely chosen strip width buys occupancy: the large-tile plan would leave at least a fifth more of the chip
// idle than the channel-major plan (the 3x3 layers with 12544 pixels and 256 filters: 98 tiles on 148 SMs against 144
// strips of 128 channels x 176 pixels; measured 8.6 -> 7.7 us and 11.4 -> 9.6 us), on problems with enough K per tile for that to
// matter and too small for the 256 x 256 pair kernel.
static bool swap_wanted(bool conv, int M, int N, int K, int num_kb, int num_iters, int num_kblocks, int cb, int sm_count) {
    if (g_path_mode >= 4 || g_swap == 2) return true;
    if (!g_swap || g_path_mode != 0 || g_force_bn >= 0) return false;
    if (N < 256 || num_iters < 8) return false;
    if (!conv && recorded_plan(M, N, K)) return false;      // a schedule recorded for this shape's class takes precedence
    const TcPlan old_plan = plan_tc(conv, M, N, K, num_kb, num_iters, num_kblocks, cb, sm_count);
    if (old_plan.two_sm || 2 * old_plan.num_tiles < sm_count) return false;   // tiny problems: launch latency, not occupancy, bounds them
    const SwapPlan sp = plan_swap_auto(M, N, num_iters, sm_count);
    if (!sp.pw) return false;
    const int waves_old = (old_plan.num_tiles + sm_count - 1) / sm_count;
    const double eff_old = (double)old_plan.num_tiles / ((double)waves_old * sm_count);
    const int workers = sp.two_sm ? sm_count / 2 : sm_count, waves_new = (sp.num_tiles + workers - 1) / workers;
    const double eff_new = (double)sp.num_tiles / ((double)waves_new * workers);
    return eff_new - eff_old >= 0.2;
}

static int run_gemm_swap(DeviceCtx* ctx, const int8_t* A, int64_t lda, const int8_t* B, int64_t ldb, int8_t* C, int64_t ldc,
                         const int32_t* bias, const int32_t* mult, const int32_t* shift, int per_channel, int M, int N, int K,
                         int relu, cudaStream_t st, const float* fscale) {
    const KLoop kl = gemm_kloop(K);
    const SwapPlan pl = plan_swap_auto(M, N, kl.num_iters, ctx->sm_count);
    if (!pl.pw || pl.stages < 2) return I8_ERR_UNSUPPORTED;
    CUtensorMap tmX;
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
    const uint64_t str[1] = {(uint64_t)lda};
    const uint32_t box[2] = {BK, (uint32_t)pl.b_rows};
    int rc = make_tmap(&tmX, A, 2, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
    return run_swap(ctx, false, pl, tmX, kl, B, ldb, C, ldc, bias, mult, shift, per_channel, M, N, K, relu, st, fscale);
}

// Implicit-GEMM convolution: A tiles come from an im2col-mode tensor map over the NHWC activations.
static int run_conv_tc(DeviceCtx* ctx, const int8_t* x, const int8_t* w, int8_t* y, const int32_t* bias, const int32_t* mult,
                       const int32_t* shift, int per_channel, int N, int H, int W, int C, int Kf, int R, int S, int P, int Q,
                       int stride_h, int stride_w, int pad_h, int pad_w, int relu, cudaStream_t st) {
    const int cb = C % 128 == 0 ? 128 : (C % 64 == 0 ? 64 : 32);
    const int M = N * P * Q;
    KLoop kl{};
    kl.cb = cb; kl.nsub = BK / cb; kl.cblocks = C / cb; kl.num_kblocks = R * S * kl.cblocks;
    kl.P = P; kl.Q = Q; kl.S = S;
    kl.inv_pq = P * Q == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)(P * Q));
    kl.inv_q = Q == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)Q);
    kl.num_iters = (kl.num_kblocks + kl.nsub - 1) / kl.nsub;
    kl.mmas_last = (kl.num_kblocks - (kl.num_iters - 1) * kl.nsub) * (cb / 32);
    kl.stride_h = stride_h; kl.stride_w = stride_w; kl.pad_h = pad_h; kl.pad_w = pad_w;
    const int K = R * S * C;
    t_used_swap = false;
    if (swap_wanted(true, M, Kf, K, (K + BK - 1) / BK, kl.num_iters, kl.num_kblocks, cb, ctx->sm_count)) {
        // filters on the tensor-memory lanes, a strip of output pixels on the columns
        const SwapPlan sp = plan_swap_auto(M, Kf, kl.num_iters, ctx->sm_count);
        if (sp.pw && sp.stages >= 2) {
            CUtensorMap tmX;
            int rc = make_tmap_im2col(&tmX, x, N, H, W, C, R, S, stride_h, stride_w, pad_h, pad_w, cb, sp.b_rows, swizzle_for(cb));
            if (rc) return rc;
            t_used_swap = true;
            return run_swap(ctx, true, sp, tmX, kl, w, K, y, Kf, bias, mult, shift, per_channel, M, Kf, K, relu, st);
        }
    }
    CUtensorMap tmA;
    {
        int rc = make_tmap_im2col(&tmA, x, N, H, W, C, R, S, stride_h, stride_w, pad_h, pad_w, cb, BM, swizzle_for(cb));
        if (rc) return rc;
    }
    // CTA pairs for convolutions follow the same measured rule as for GEMMs, or are asked for explicitly (path mode 2, I8OPS_CONV2SM=1)
    const TcPlan pl = plan_tc(true, M, Kf, K, (K + BK - 1) / BK, kl.num_iters, kl.num_kblocks, cb, ctx->sm_count);
    return run_tc(ctx, true, pl, tmA, kl, w, K, y, Kf, bias, mult, shift, per_channel, M, Kf, K, relu, st);
}

// Stream-ordered workspaces: a memory pool the library creates per device on first use.  A block is allocated on the
// caller's stream before the launches that use it and released behind them (release threshold unlimited, so the next call
// reuses it): concurrent streams never share a block, the calls stay asynchronous, and a captured graph owns its copy.
static const int64_t WORKSPACE_MAX_BYTES = 256ll << 20;
static int pool_alloc(DeviceCtx* ctx, void** out, int64_t bytes, cudaStream_t st) {
    if (bytes <= 0 || bytes > WORKSPACE_MAX_BYTES) return I8_ERR_UNSUPPORTED;
    if (!ctx->pool_ready.load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (!ctx->pool_ready.load(std::memory_order_relaxed)) {
            int dev = 0;
            CUDA_TRY(cudaGetDevice(&dev));
            cudaMemPoolProps props{};
            props.allocType = cudaMemAllocationTypePinned;
            props.handleTypes = cudaMemHandleTypeNone;
            props.location.type = cudaMemLocationTypeDevice;
            props.location.id = dev;
            if (cudaMemPoolCreate(&ctx->pool, &props) != cudaSuccess) { cudaGetLastError(); return I8_ERR_UNSUPPORTED; }
            uint64_t keep = ~0ull;
            cudaMemPoolSetAttribute(ctx->pool, cudaMemPoolAttrReleaseThreshold, &keep);
            ctx->pool_ready.store(true, std::memory_order_release);
        }
    }
    if (cudaMallocFromPoolAsync(out, (size_t)bytes, ctx->pool, st) != cudaSuccess) { cudaGetLastError(); return I8_ERR_UNSUPPORTED; }
    return I8_OK;
}

static int grid_for(int64_t items) {
    int64_t blocks = (items + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    return (int)(blocks < 1 ? 1 : blocks);
}

static int launch_pack(const int8_t* src, int64_t rs, int64_t cs, int rows, int K, int kp, int8_t* dst, cudaStream_t st) {
    PackParams pk{src, dst, rs, cs, rows, K, kp};
    pack_rows_i8_kernel<<<grid_for((int64_t)rows * (kp / 16)), 256, 0, st>>>(pk);
    const cudaError_t le = cudaGetLastError();
    return le == cudaSuccess ? I8_OK : cuda_fail(le);
}

static int64_t up256(int64_t v) { return (v + 255) & ~(int64_t)255; }

// Convolutions the im2col tensor maps do not take (small activation tensors, long strides, large filters, channel counts
// that are not a multiple of 32): the activations are unfolded into the GEMM form's A matrix in a stream-ordered
// workspace, then the product runs on the tensor path.  With C % 16 != 0 the rows of that matrix and of a repacked copy
// of the filters are padded with zeros to a multiple of 16 bytes.  Returns I8_ERR_UNSUPPORTED, launching nothing, when
// the workspace would be too large or cannot be had.
static int run_conv_unfold(DeviceCtx* ctx, const int8_t* x, const int8_t* w, int8_t* y, const int32_t* bias, const int32_t* mult,
                           const int32_t* shift, int per_channel, int N, int H, int W, int C, int Kf, int R, int S, int P, int Q,
                           int stride_h, int stride_w, int pad_h, int pad_w, int relu, cudaStream_t st) {
    const int64_t M = (int64_t)N * P * Q, K = (int64_t)R * S * C;
    if (M >= (1ll << 31)) return I8_ERR_UNSUPPORTED;
    const bool whole_pieces = C % 16 == 0 && aligned16(x) && aligned16(w);
    const int64_t kp = (K + 15) & ~(int64_t)15;
    const int64_t a_bytes = up256(M * kp), w_bytes = whole_pieces ? 0 : up256((int64_t)Kf * kp);
    void* ws = nullptr;
    int rc = pool_alloc(ctx, &ws, a_bytes + w_bytes, st);
    if (rc) return rc;
    int8_t* a = (int8_t*)ws;
    const int8_t* wmat = w;
    cudaError_t le;
    if (whole_pieces) {
        UnfoldParams u{x, a, N, H, W, C, R, S, P, Q, stride_h, stride_w, pad_h, pad_w};
        conv_unfold_i8_kernel<<<grid_for(M * K / 16), 256, 0, st>>>(u);
        le = cudaGetLastError();
    } else {
        UnfoldBytesParams u{x, a, N, H, W, C, R, S, P, Q, stride_h, stride_w, pad_h, pad_w, (int)kp};
        conv_unfold_bytes_i8_kernel<<<grid_for(M * (kp / 16)), 256, 0, st>>>(u);
        le = cudaGetLastError();
        if (le == cudaSuccess) {
            rc = launch_pack(w, K, 1, Kf, (int)K, (int)kp, a + a_bytes, st);
            wmat = a + a_bytes;
        }
    }
    if (le != cudaSuccess) rc = cuda_fail(le);
    if (rc == I8_OK) {
        t_used_two_sm = false; t_tmap_failed = false;
        rc = run_gemm_tc(ctx, a, kp, wmat, kp, y, Kf, bias, mult, shift, per_channel, (int)M, Kf, (int)kp, relu, st);
    }
    cudaFreeAsync(ws, st);
    return rc;
}

// GEMM operands the tensor path cannot fetch in place (a base or leading dimension that is not a multiple of 16 bytes,
// general strides): packed into K-contiguous, zero-padded copies in a stream-ordered workspace, then the tensor path.
// Operands that are already in a legal layout are used where they are.
static int run_gemm_packed(DeviceCtx* ctx, const int8_t* A, int64_t a_rs, int64_t a_cs, bool a_ok, const int8_t* B, int64_t b_rs,
                           int64_t b_cs, bool b_ok, int8_t* C, int64_t ldc, const int32_t* bias, const int32_t* mult,
                           const int32_t* shift, int per_channel, int M, int N, int K, int relu, cudaStream_t st,
                           const RawOut& raw = RawOut(), const float* fscale = nullptr) {
    const int64_t kp = ((int64_t)K + 15) & ~(int64_t)15;
    const int64_t a_bytes = a_ok ? 0 : up256((int64_t)M * kp), b_bytes = b_ok ? 0 : up256((int64_t)N * kp);
    void* ws = nullptr;
    int rc = pool_alloc(ctx, &ws, a_bytes + b_bytes, st);
    if (rc) return rc;
    const int8_t* Ap = A; int64_t lda = a_rs;
    const int8_t* Bp = B; int64_t ldb = b_cs;
    if (!a_ok) {
        rc = launch_pack(A, a_rs, a_cs, M, K, (int)kp, (int8_t*)ws, st);
        Ap = (int8_t*)ws; lda = kp;
    }
    if (rc == I8_OK && !b_ok) {
        rc = launch_pack(B, b_cs, b_rs, N, K, (int)kp, (int8_t*)ws + a_bytes, st);      // row n of the copy = column n of B
        Bp = (int8_t*)ws + a_bytes; ldb = kp;
    }
    if (rc == I8_OK) {
        t_used_two_sm = false; t_tmap_failed = false;
        if (fscale) {
            rc = run_gemm_swap(ctx, Ap, lda, Bp, ldb, C, ldc, bias, nullptr, nullptr, per_channel, M, N, K, relu, st, fscale);
            if (rc == I8_OK) t_used_swap = true;
        } else {
            rc = run_gemm_tc(ctx, Ap, lda, Bp, ldb, C, ldc, bias, mult, shift, per_channel, M, N, K, relu, st, raw);
        }
    }
    cudaFreeAsync(ws, st);
    return rc;
}

// Slab-resident stride-1 convolution (conv_slab.cuh): plan and launch.  Returns I8_ERR_UNSUPPORTED, launching nothing,
// when the layer does not fit the kernel (the caller then takes the implicit-GEMM path).
static int run_conv_slab(DeviceCtx* ctx, const int8_t* x, const int8_t* w, int8_t* y, const int32_t* bias, const int32_t* mult,
                         const int32_t* shift, int per_channel, int N, int H, int W, int C, int Kf, int R, int S, int P, int Q,
                         int pad_h, int pad_w, int relu, cudaStream_t st) {
    const int Wp = W + 2 * pad_w;
    if (C % 32 != 0 || Wp > BM || Kf > 128 || R * S > 49 || Q < 1 || P < 1) return I8_ERR_UNSUPPORTED;
    const int TH = BM / Wp;
    const int slab_rows = TH + R - 1;
    if (slab_rows > 256 || 2 * TH * Q < BM) return I8_ERR_UNSUPPORTED;        // at least half of the 128 lanes must be real outputs
    const int bn = Kf <= 64 ? 64 : 128;
    const int cb = C % 128 == 0 ? 128 : (C % 64 == 0 ? 64 : 32);
    const int cblocks = C / cb;
    const int64_t tiles_per_img = (P + TH - 1) / TH;
    if ((int64_t)N * tiles_per_img >= (1ll << 30)) return I8_ERR_UNSUPPORTED;
    auto up1k = [](int64_t v) { return (v + 1023) & ~(int64_t)1023; };
    const int64_t slab_tx = (int64_t)cb * Wp * slab_rows;
    const int64_t reach = (int64_t)(BM + (R - 1) * Wp + S - 1) * cb;          // furthest byte any tap's 128 rows touch
    const int64_t stage_bytes = up1k(slab_tx > reach ? slab_tx : reach);
    const int64_t w_bytes = (int64_t)R * S * C * bn;                           // resident filter bank, zero rows up to bn
    const int64_t fixed = up1k(w_bytes) + 9 * bn * 4 + (2 * SLAB_MAX_STAGES + 2 * SLAB_ACC + 1) * 8 + 16;
    const int64_t budget = 227 * 1024 - 1024;
    int64_t stages = (budget - fixed) / stage_bytes;
    if (stages > SLAB_MAX_STAGES) stages = SLAB_MAX_STAGES;
    if (stages < 2) return I8_ERR_UNSUPPORTED;
    CUtensorMap tmX, tmW;
    {
        const uint64_t dims[4] = {(uint64_t)C, (uint64_t)W, (uint64_t)H, (uint64_t)N};
        const uint64_t str[3] = {(uint64_t)C, (uint64_t)W * C, (uint64_t)H * W * C};
        const uint32_t box[4] = {(uint32_t)cb, (uint32_t)Wp, (uint32_t)slab_rows, 1};
        int rc = make_tmap(&tmX, x, 4, dims, str, box, swizzle_for(cb));
        if (rc) return rc;
    }
    {
        const uint64_t dims[2] = {(uint64_t)R * S * C, (uint64_t)Kf};
        const uint64_t str[1] = {(uint64_t)R * S * C};
        const uint32_t box[2] = {(uint32_t)cb, (uint32_t)bn};
        int rc = make_tmap(&tmW, w, 2, dims, str, box, swizzle_for(cb));
        if (rc) return rc;
    }
    ConvSlabParams p;
    p.y = y; p.bias = bias; p.mult = mult; p.shift = shift; p.per_channel = per_channel; p.relu = relu;
    p.Kf = Kf; p.P = P; p.Q = Q; p.R = R; p.S = S; p.Wp = Wp; p.TH = TH; p.pad_h = pad_h; p.pad_w = pad_w;
    p.cb = cb; p.cblocks = cblocks;
    p.tiles_per_img = (int)tiles_per_img; p.num_tiles = (int)(N * tiles_per_img);
    p.inv_tpi = tiles_per_img == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)tiles_per_img);
    p.inv_wp = Wp == 1 ? 0xffffffffu : (uint32_t)((1ull << 32) / (uint64_t)Wp);
    p.slab_tx_bytes = (int)slab_tx; p.stage_bytes = (int)stage_bytes; p.stages = (int)stages;
    p.off_b = (int)(stages * stage_bytes);
    p.off_const = p.off_b + (int)up1k(w_bytes);
    p.off_bar = p.off_const + 9 * bn * 4;
    p.y_vec_ok = aligned16(y) && Kf % 16 == 0;
    p.wait_limit_cycles = (long long)(g_wait_limit_ns * 2);
    p.dev_status = ctx->dev_status;
    const size_t smem = (size_t)p.off_bar + (2 * SLAB_MAX_STAGES + 2 * SLAB_ACC + 1) * 8 + 16 + 1024;
    const int grid = p.num_tiles < ctx->sm_count ? p.num_tiles : ctx->sm_count;
    // 3 x 3 filters get the instance whose issue loop is unrolled over the nine taps
    void (*kern)(CUtensorMap, CUtensorMap, ConvSlabParams);
    int slot;
    if (R == 3 && S == 3) { kern = bn == 64 ? conv_slab_i8_kernel<64, 9> : conv_slab_i8_kernel<128, 9>; slot = bn == 64 ? 11 : 12; }
    else { kern = bn == 64 ? conv_slab_i8_kernel<64, 0> : conv_slab_i8_kernel<128, 0>; slot = bn == 64 ? 13 : 14; }
    if (!ctx->attr_set[slot]) {
        CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        ctx->attr_set[slot] = true;
    }
    CUDA_TRY(launch_kernel(kern, true, 1, grid, SLAB_THREADS, smem, st, tmX, tmW, p));
    return I8_OK;
}

// Paired small-tile path: problems with M, N, K <= 64, two per MMA.
static int run_batched_pair(DeviceCtx* ctx, const int8_t* A, int64_t a_rs, int64_t a_bs, const int8_t* B, int64_t b_ld,
                            int64_t b_bs, int b_mn_major, int8_t* C, int64_t ldc, int64_t c_bs, const int32_t* bias,
                            int64_t bias_bs, const int32_t* mult, const int32_t* shift, int per_channel, int batch, int M,
                            int N, int K, int relu, cudaStream_t st) {
    CUtensorMap tmA, tmB;
    const uint32_t box[3] = {64, 64, 2};
    {
        const uint64_t dims[3] = {(uint64_t)K, (uint64_t)M, (uint64_t)batch};
        const uint64_t str[2] = {(uint64_t)a_rs, (uint64_t)a_bs};
        int rc = make_tmap(&tmA, A, 3, dims, str, box, CU_TENSOR_MAP_SWIZZLE_64B);
        if (rc) return rc;
    }
    {
        const uint64_t dimsK[3] = {(uint64_t)K, (uint64_t)N, (uint64_t)batch};   // K contiguous: rows are output columns
        const uint64_t dimsN[3] = {(uint64_t)N, (uint64_t)K, (uint64_t)batch};   // N contiguous: rows are K
        const uint64_t str[2] = {(uint64_t)b_ld, (uint64_t)b_bs};
        int rc = make_tmap(&tmB, B, 3, b_mn_major ? dimsN : dimsK, str, box, CU_TENSOR_MAP_SWIZZLE_64B);
        if (rc) return rc;
    }
    BatchedPairParams p;
    p.C = C; p.ldc = ldc; p.c_bs = c_bs; p.bias = bias; p.bias_bs = bias_bs; p.mult = mult; p.shift = shift;
    p.per_channel = per_channel; p.relu = relu; p.batch = batch; p.M = M; p.N = N; p.K = K;
    p.b_mn_major = b_mn_major;
    p.c_vec_ok = aligned16(C) && ldc % 16 == 0 && c_bs % 16 == 0;
    p.bias_vec_ok = bias && aligned16(bias) && bias_bs % 4 == 0;
    p.wait_limit_cycles = (long long)(g_wait_limit_ns * 2);
    p.dev_status = ctx->dev_status;
    if (!ctx->attr_set[6]) {
        CUDA_TRY(cudaFuncSetAttribute(batched_pair_i8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PairSmem::DYN_BYTES));
        ctx->attr_set[6] = true;
    }
    const int pairs = (batch + 1) / 2;
    const int grid = pairs < ctx->sm_count ? pairs : ctx->sm_count;
    CUDA_TRY(launch_kernel(batched_pair_i8_kernel, true, 1, grid, PAIR_THREADS, PairSmem::DYN_BYTES, st, tmA, tmB, p));
    return I8_OK;
}

static int run_gemm_generic(const GenericGemmParams& p, cudaStream_t st) {
    const int64_t total = (int64_t)p.batch * p.M * p.N;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    gemm_i8_generic_kernel<<<(int)blocks, 256, 0, st>>>(p);
    CUDA_TRY(cudaGetLastError());
    return I8_OK;
}

// One operand's strides: the unit stride picks the contiguous axis, the other must span it.
static bool strides_ok(int64_t rs, int64_t cs, int rows, int cols) {
    if (rs < 0 || cs < 0) return false;
    if (cs == 1 && (rs >= cols || rows <= 1)) return true;
    if (rs == 1 && (cs >= rows || cols <= 1)) return true;
    return false;
}

static int validate_gemm(const void* A, int64_t a_rs, int64_t a_cs, const void* B, int64_t b_rs, int64_t b_cs, const void* C,
                         int64_t ldc, const void* mult, const void* shift, int M, int N, int K) {
    if (M < 0 || N < 0 || K < 0) return I8_ERR_SHAPE;
    if (K > 65536) return I8_ERR_RANGE;
    if (M == 0 || N == 0) return I8_OK;
    if (!C || !mult || !shift || (K > 0 && (!A || !B))) return I8_ERR_NULL;
    if (!strides_ok(a_rs, a_cs, M, K) || !strides_ok(b_rs, b_cs, K, N)) return I8_ERR_STRIDE;
    if (ldc < N) return I8_ERR_STRIDE;
    return I8_OK;
}

}  // namespace i8

using namespace i8;

// ================================================================================================ C ABI
extern "C" {

int gemm_i8(const int8_t* A, int64_t a_rs, int64_t a_cs, const int8_t* B, int64_t b_rs, int64_t b_cs, int8_t* C, int64_t ldc,
            const int32_t* bias, const int32_t* mult, const int32_t* shift, int per_channel, int M, int N, int K, int relu,
            void* stream) {
    t_last_path = I8_PATH_NONE;
    t_last_packed = false;
    int rc = validate_gemm(A, a_rs, a_cs, B, b_rs, b_cs, C, ldc, mult, shift, M, N, K);
    if (rc) return rc;
    if (M == 0 || N == 0) return I8_OK;
    DeviceCtx* ctx = nullptr;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // the tensor path takes either storage order of either operand: K contiguous (K-major) or M / N contiguous
    const bool a_k = a_cs == 1 && a_rs % 16 == 0 && a_rs >= K, a_m = !a_k && a_rs == 1 && a_cs % 16 == 0 && a_cs >= M;
    const bool b_k = b_rs == 1 && b_cs % 16 == 0 && b_cs >= K, b_n = !b_k && b_cs == 1 && b_rs % 16 == 0 && b_rs >= N;
    const bool tc_legal = K >= 1 && aligned16(A) && aligned16(B) && (a_k || a_m) && (b_k || b_n);
    if (tc_legal && g_path_mode != 1) {
        t_used_two_sm = false; t_tmap_failed = false;
        rc = run_gemm_tc(ctx, A, a_k ? a_rs : a_cs, B, b_k ? b_cs : b_rs, C, ldc, bias, mult, shift, per_channel, M, N, K, relu, st, RawOut(),
                         a_m ? 1 : 0, b_n ? 1 : 0);
        if (rc == I8_OK) t_last_path = tensor_path_used();
        if (!(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
        // the driver refused a tensor map for this geometry: nothing was launched, the generic kernel serves it
    } else if (g_path_mode != 1 && g_unfold && K >= 1 && (int64_t)M * N * K >= (1ll << 18)) {
        // operands the tensor path cannot fetch in place: packed copies in a stream-ordered workspace (tiny problems are
        // quicker on the generic kernel than behind two extra launches)
        rc = run_gemm_packed(ctx, A, a_rs, a_cs, a_k && aligned16(A), B, b_rs, b_cs, b_k && aligned16(B), C, ldc, bias, mult, shift,
                             per_channel, M, N, K, relu, st);
        if (rc == I8_OK) { t_last_path = tensor_path_used(); t_last_packed = true; return rc; }
        if (rc != I8_ERR_UNSUPPORTED && !(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
    }
    GenericGemmParams g{A, a_rs, a_cs, 0, B, b_rs, b_cs, 0, C, ldc, 0, bias, 0, mult, shift, per_channel, relu, 1, M, N, K, nullptr, 0, 0, 0};
    rc = run_gemm_generic(g, st);
    if (rc == I8_OK) t_last_path = I8_PATH_GENERIC;
    return rc;
}

int gemm_i8_raw(const int8_t* A, int64_t a_rs, int64_t a_cs, const int8_t* B, int64_t b_rs, int64_t b_cs, int32_t* D, int64_t ldd,
                int accumulate, int M, int N, int K, void* stream) {
    t_last_path = I8_PATH_NONE;
    t_last_packed = false;
    if (M < 0 || N < 0 || K < 0) return I8_ERR_SHAPE;
    if (K > 65536) return I8_ERR_RANGE;
    if (M == 0 || N == 0) return I8_OK;
    if (!D || (K > 0 && (!A || !B))) return I8_ERR_NULL;
    if (!strides_ok(a_rs, a_cs, M, K) || !strides_ok(b_rs, b_cs, K, N) || ldd < N) return I8_ERR_STRIDE;
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // the tensor path takes either storage order of either operand: K contiguous (K-major) or M / N contiguous
    const bool a_k = a_cs == 1 && a_rs % 16 == 0 && a_rs >= K, a_m = !a_k && a_rs == 1 && a_cs % 16 == 0 && a_cs >= M;
    const bool b_k = b_rs == 1 && b_cs % 16 == 0 && b_cs >= K, b_n = !b_k && b_cs == 1 && b_rs % 16 == 0 && b_rs >= N;
    const bool tc_legal = K >= 1 && aligned16(A) && aligned16(B) && (a_k || a_m) && (b_k || b_n);
    if (tc_legal && g_path_mode != 1) {
        RawOut raw; raw.D = D; raw.ldd = ldd; raw.accumulate = accumulate ? 1 : 0;
        t_used_two_sm = false; t_tmap_failed = false;
        rc = run_gemm_tc(ctx, A, a_k ? a_rs : a_cs, B, b_k ? b_cs : b_rs, nullptr, 0, nullptr, nullptr, nullptr, 0, M, N, K, 0, st, raw,
                         a_m ? 1 : 0, b_n ? 1 : 0);
        if (rc == I8_OK) t_last_path = tensor_path_used();
        if (!(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
    } else if (g_path_mode != 1 && g_unfold && K >= 1 && (int64_t)M * N * K >= (1ll << 18)) {
        RawOut raw; raw.D = D; raw.ldd = ldd; raw.accumulate = accumulate ? 1 : 0;
        rc = run_gemm_packed(ctx, A, a_rs, a_cs, a_k && aligned16(A), B, b_rs, b_cs, b_k && aligned16(B), nullptr, 0, nullptr, nullptr,
                             nullptr, 0, M, N, K, 0, st, raw);
        if (rc == I8_OK) { t_last_path = tensor_path_used(); t_last_packed = true; return rc; }
        if (rc != I8_ERR_UNSUPPORTED && !(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
    }
    GenericGemmParams g{A, a_rs, a_cs, 0, B, b_rs, b_cs, 0, nullptr, 0, 0, nullptr, 0, nullptr, nullptr, 0, 0, 1, M, N, K,
                        D, ldd, 1, accumulate ? 1 : 0};
    rc = run_gemm_generic(g, st);
    if (rc == I8_OK) t_last_path = I8_PATH_GENERIC;
    return rc;
}

int gemm_i8_fscale(const int8_t* A, int64_t a_rs, int64_t a_cs, const int8_t* B, int64_t b_rs, int64_t b_cs, int8_t* C, int64_t ldc,
                   const int32_t* bias, const float* scale, int per_channel, int M, int N, int K, int relu, void* stream) {
    t_last_path = I8_PATH_NONE;
    t_last_packed = false;
    if (M < 0 || N < 0 || K < 0) return I8_ERR_SHAPE;
    if (K > 65536) return I8_ERR_RANGE;
    if (M == 0 || N == 0) return I8_OK;
    if (!C || !scale || (K > 0 && (!A || !B))) return I8_ERR_NULL;
    if (!strides_ok(a_rs, a_cs, M, K) || !strides_ok(b_rs, b_cs, K, N) || ldc < N) return I8_ERR_STRIDE;
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // tensor path: the channel-major kernel (every thread owns one output channel, so the scale is one register)
    const bool tc_legal = K >= 1 && a_cs == 1 && b_rs == 1 && aligned16(A) && aligned16(B) && a_rs % 16 == 0 && b_cs % 16 == 0 &&
                          a_rs >= K && b_cs >= K;
    if (tc_legal && g_path_mode != 1) {
        t_used_two_sm = false; t_tmap_failed = false;
        rc = run_gemm_swap(ctx, A, a_rs, B, b_cs, C, ldc, bias, nullptr, nullptr, per_channel, M, N, K, relu, st, scale);
        if (rc == I8_OK) { t_used_swap = true; t_last_path = tensor_path_used(); return rc; }
        if (rc != I8_ERR_UNSUPPORTED && !(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
    } else if (g_path_mode != 1 && g_unfold && K >= 1 && (int64_t)M * N * K >= (1ll << 18)) {
        // misaligned or M- / N-contiguous operands: packed K-contiguous copies, then the channel-major kernel
        const bool a_ok = a_cs == 1 && a_rs % 16 == 0 && a_rs >= K && aligned16(A), b_ok = b_rs == 1 && b_cs % 16 == 0 && b_cs >= K && aligned16(B);
        t_used_two_sm = false; t_tmap_failed = false;
        rc = run_gemm_packed(ctx, A, a_rs, a_cs, a_ok, B, b_rs, b_cs, b_ok, C, ldc, bias, nullptr, nullptr, per_channel, M, N, K, relu, st,
                             RawOut(), scale);
        if (rc == I8_OK) { t_last_path = tensor_path_used(); t_last_packed = true; return rc; }
        if (rc != I8_ERR_UNSUPPORTED && !(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
    }
    GenericGemmParams g{A, a_rs, a_cs, 0, B, b_rs, b_cs, 0, C, ldc, 0, bias, 0, nullptr, nullptr, per_channel, relu, 1, M, N, K,
                        nullptr, 0, 0, 0, scale};
    rc = run_gemm_generic(g, st);
    if (rc == I8_OK) t_last_path = I8_PATH_GENERIC;
    return rc;
}

int batched_gemm_i8(const int8_t* A, int64_t a_rs, int64_t a_cs, int64_t a_bs, const int8_t* B, int64_t b_rs, int64_t b_cs,
                    int64_t b_bs, int8_t* C, int64_t ldc, int64_t c_bs, const int32_t* bias, int64_t bias_bs,
                    const int32_t* mult, const int32_t* shift, int per_channel, int batch, int M, int N, int K, int relu,
                    void* stream) {
    t_last_path = I8_PATH_NONE;
    if (batch < 0) return I8_ERR_SHAPE;
    int rc = validate_gemm(A, a_rs, a_cs, B, b_rs, b_cs, C, ldc, mult, shift, M, N, K);
    if (rc) return rc;
    if (a_bs < 0 || b_bs < 0 || c_bs < 0 || bias_bs < 0) return I8_ERR_STRIDE;
    if (batch == 0 || M == 0 || N == 0) return I8_OK;
    DeviceCtx* ctx = nullptr;
    rc = get_ctx(&ctx);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // (an operand shared by all problems, batch stride 0, has no 3-D tensor map: the generic kernel serves it)
    if (g_path_mode != 1 && M <= 64 && N <= 64 && K >= 1 && K <= 64 && a_cs == 1 && aligned16(A) && aligned16(B) &&
        a_rs % 16 == 0 && a_bs % 16 == 0 && b_bs % 16 == 0 && a_rs >= K && (batch == 1 || (a_bs > 0 && b_bs > 0))) {
        const bool b_n_contig = b_cs == 1 && b_rs % 16 == 0 && b_rs >= N;      // row-major B: MN-major operand
        const bool b_k_contig = b_rs == 1 && b_cs % 16 == 0 && b_cs >= K;      // column-major B: K-major operand
        if (b_k_contig || b_n_contig) {
            t_tmap_failed = false;
            rc = run_batched_pair(ctx, A, a_rs, a_bs, B, b_k_contig ? b_cs : b_rs, b_bs, b_k_contig ? 0 : 1, C, ldc, c_bs,
                                  bias, bias_bs, mult, shift, per_channel, batch, M, N, K, relu, st);
            if (rc == I8_OK) t_last_path = I8_PATH_SMALL;
            if (!(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
        }
    }
    // Larger problems with aligned slices.  All problems in ONE launch of the large-tile kernel when A is K-contiguous and
    // the batch strides are whole rows (the tile schedule runs over the stacked problems); otherwise one launch per
    // problem, when each problem is big enough to be worth a launch of its own (128^3 multiply-accumulates, or a short
    // batch).
    if (g_path_mode != 1 && K >= 1 && batch <= 65536) {
        const bool a_k = a_cs == 1 && a_rs % 16 == 0 && a_rs >= K, a_m = !a_k && a_rs == 1 && a_cs % 16 == 0 && a_cs >= M;
        const bool b_k = b_rs == 1 && b_cs % 16 == 0 && b_cs >= K, b_n = !b_k && b_cs == 1 && b_rs % 16 == 0 && b_rs >= N;
        if (aligned16(A) && aligned16(B) && a_bs % 16 == 0 && b_bs % 16 == 0 && (a_k || a_m) && (b_k || b_n)) {
            if (batch > 1 && a_k && a_bs > 0 && b_bs > 0 && c_bs > 0) {
                t_used_two_sm = false; t_tmap_failed = false; t_used_swap = false;
                rc = run_gemm_tc_batched(ctx, A, a_rs, a_bs, B, b_k ? b_cs : b_rs, b_bs, C, ldc, c_bs, bias, bias_bs, mult, shift,
                                         per_channel, batch, M, N, K, relu, st, b_n ? 1 : 0);
                if (rc == I8_OK) { t_last_path = tensor_path_used(); return rc; }
                if (rc != I8_ERR_UNSUPPORTED && !(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
            }
            if ((int64_t)M * N * K >= (1ll << 21) || batch <= 8) {
                int last = I8_PATH_NONE;
                for (int b = 0; b < batch; b++) {
                    t_used_two_sm = false; t_tmap_failed = false;
                    rc = run_gemm_tc(ctx, A + (int64_t)b * a_bs, a_k ? a_rs : a_cs, B + (int64_t)b * b_bs, b_k ? b_cs : b_rs, C + (int64_t)b * c_bs, ldc,
                                     bias ? bias + (int64_t)b * bias_bs : nullptr, mult, shift, per_channel, M, N, K, relu, st, RawOut(),
                                     a_m ? 1 : 0, b_n ? 1 : 0);
                    if (rc == I8_ERR_CUDA && t_tmap_failed && b == 0) break;        // no tensor map for this geometry: generic kernel below
                    if (rc) return rc;
                    last = tensor_path_used();
                }
                if (rc == I8_OK) { t_last_path = last; return rc; }
            }
        }
    }
    GenericGemmParams g{A, a_rs, a_cs, a_bs, B, b_rs, b_cs, b_bs, C, ldc, c_bs, bias, bias_bs, mult, shift, per_channel, relu,
                        batch, M, N, K, nullptr, 0, 0, 0};
    rc = run_gemm_generic(g, st);
    if (rc == I8_OK) t_last_path = I8_PATH_GENERIC;
    return rc;
}

int conv2d_i8(const int8_t* x, const int8_t* w, int8_t* y, const int32_t* bias, const int32_t* mult, const int32_t* shift,
              int per_channel, int N, int H, int W, int C, int K, int R, int S, int stride_h, int stride_w, int pad_h,
              int pad_w, int relu, void* stream) {
    t_last_path = I8_PATH_NONE;
    t_last_unfold = false;
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || K <= 0 || R <= 0 || S <= 0) return I8_ERR_SHAPE;
    if (stride_h < 1 || stride_w < 1 || pad_h < 0 || pad_w < 0) return I8_ERR_UNSUPPORTED;
    if (H + 2 * pad_h < R || W + 2 * pad_w < S) return I8_ERR_SHAPE;
    if ((int64_t)R * S * C > 65536) return I8_ERR_RANGE;
    if (!x || !w || !y || !mult || !shift) return I8_ERR_NULL;
    const int P = (H + 2 * pad_h - R) / stride_h + 1;
    const int Q = (W + 2 * pad_w - S) / stride_w + 1;
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (g_path_mode != 1 && aligned16(x) && aligned16(w)) {
        if (R == 1 && S == 1 && stride_h == 1 && stride_w == 1 && pad_h == 0 && pad_w == 0 && C % 16 == 0 &&
            (int64_t)N * H * W < (1ll << 31)) {
            // a 1x1 convolution is the GEMM [N*H*W, C] x [C, K]
            t_used_two_sm = false; t_tmap_failed = false;
            rc = run_gemm_tc(ctx, x, C, w, C, y, K, bias, mult, shift, per_channel, N * H * W, K, C, relu, st);
            if (rc == I8_OK) t_last_path = tensor_path_used();
            if (!(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
        }
        if (g_slab && g_path_mode == 0 && stride_h == 1 && stride_w == 1 && (int64_t)N * P * Q < (1ll << 31)) {
            // few filters and a narrow image: keep the input slab in shared memory and reuse it across the filter taps
            t_tmap_failed = false;
            rc = run_conv_slab(ctx, x, w, y, bias, mult, shift, per_channel, N, H, W, C, K, R, S, P, Q, pad_h, pad_w, relu, st);
            if (rc == I8_OK) { t_last_path = I8_PATH_CONV_SLAB; return rc; }
            if (rc != I8_ERR_UNSUPPORTED && !(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
        }
        // im2col tensor maps: channel blocks of 32/64/128 bytes, box corners and tap offsets within the 4-D
        // encoding's ranges, traversal strides up to 8; activation tensors below 128 KiB stay on the generic kernel
        const bool tc_legal = C % 32 == 0 && R <= 16 && S <= 16 && pad_h <= 16 && pad_w <= 16 && stride_h <= 8 &&
                              stride_w <= 8 && (int64_t)N * H * W * C >= 131072 && (int64_t)N * P * Q < (1ll << 31);
        if (tc_legal) {
            t_used_two_sm = false; t_tmap_failed = false;
            rc = run_conv_tc(ctx, x, w, y, bias, mult, shift, per_channel, N, H, W, C, K, R, S, P, Q, stride_h, stride_w,
                             pad_h, pad_w, relu, st);
            if (rc == I8_OK) t_last_path = tensor_path_used();
            if (!(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
        }
    }
    if (g_path_mode != 1 && g_unfold) {
        rc = run_conv_unfold(ctx, x, w, y, bias, mult, shift, per_channel, N, H, W, C, K, R, S, P, Q, stride_h, stride_w,
                             pad_h, pad_w, relu, st);
        if (rc == I8_OK) { t_last_path = tensor_path_used(); t_last_unfold = true; return rc; }
        if (rc != I8_ERR_UNSUPPORTED && !(rc == I8_ERR_CUDA && t_tmap_failed)) return rc;
    }
    GenericConvParams g{x, w, y, bias, mult, shift, per_channel, relu, N, H, W, C, K, R, S, P, Q, stride_h, stride_w, pad_h, pad_w};
    const int64_t total = (int64_t)N * P * Q * K;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    conv2d_i8_generic_kernel<<<(int)blocks, 256, 0, st>>>(g);
    CUDA_TRY(cudaGetLastError());
    t_last_path = I8_PATH_GENERIC;
    return I8_OK;
}

int i8ops_last_conv_unfolded(void) { return t_last_unfold ? 1 : 0; }
int i8ops_last_gemm_packed(void) { return t_last_packed ? 1 : 0; }

int gemm_i8_host(const int8_t* A, const int8_t* B, int8_t* C, const int32_t* bias, const int32_t* mult, const int32_t* shift,
                 int per_channel, int M, int N, int K, int relu, void* stream) {
    t_last_path = I8_PATH_NONE;
    if (M < 0 || N < 0 || K < 0) return I8_ERR_SHAPE;
    if (K > 65536) return I8_ERR_RANGE;
    if (M == 0 || N == 0) return I8_OK;
    if (!C || !mult || !shift || (K > 0 && (!A || !B))) return I8_ERR_NULL;
    const int nq = per_channel ? N : 1;
    for (int i = 0; i < nq; i++)
        if (shift[i] < 0 || shift[i] > 31) return I8_ERR_RANGE;
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // One call at a time per device: the workspace, the two copy streams and the events below belong to the device's
    // context, so a second host thread waits here until the first call has synchronised and returned.
    std::lock_guard<std::mutex> host_lock(ctx->host_mutex);
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t szA = up((size_t)M * K), szB = up((size_t)N * K), szC = up((size_t)M * N);
    const size_t szV = up((size_t)N * 4);
    const size_t need = szA + szB + szC + 3 * szV;
    if (ctx->ws_bytes < need) {
        // every earlier call synchronised before it returned, so nothing still uses the old workspace
        if (ctx->ws) { CUDA_TRY(cudaFree(ctx->ws)); ctx->ws = nullptr; ctx->ws_bytes = 0; }
        CUDA_TRY(cudaMalloc(&ctx->ws, need));
        ctx->ws_bytes = need;
    }
    uint8_t* base = (uint8_t*)ctx->ws;
    int8_t* dA = (int8_t*)base; int8_t* dB = (int8_t*)(base + szA); int8_t* dC = (int8_t*)(base + szA + szB);
    int32_t* dbias = (int32_t*)(base + szA + szB + szC);
    int32_t* dmult = (int32_t*)((uint8_t*)dbias + szV);
    int32_t* dshift = (int32_t*)((uint8_t*)dmult + szV);
    // Row chunks are pipelined over three streams: copy-in of chunk i+1, the kernel on chunk i and copy-out of chunk i-1
    // overlap (the two copy directions use separate DMA engines), so the host link is busy in both directions.
    const int nchunks = (K > 0 && M >= 2048) ? (M >= 8192 ? 8 : 4) : 1;
    if (nchunks > 1 && !ctx->s_in) {
        CUDA_TRY(cudaStreamCreateWithFlags(&ctx->s_out, cudaStreamNonBlocking));
        for (auto& e : ctx->ev) CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        CUDA_TRY(cudaStreamCreateWithFlags(&ctx->s_in, cudaStreamNonBlocking));
    }
    // Whatever was queued before an error is allowed to finish before the call returns: the buffers are the caller's
    // and the workspace may be handed to the next call.
    auto drain = [&](int status) {
        if (ctx->s_in) cudaStreamSynchronize(ctx->s_in);
        if (ctx->s_out) cudaStreamSynchronize(ctx->s_out);
        cudaStreamSynchronize(st);
        return status;
    };
#define HOST_TRY(expr) do { cudaError_t _e = (expr); if (_e != cudaSuccess) return drain(cuda_fail(_e)); } while (0)
    if (nchunks == 1) {
        if (K > 0) {
            HOST_TRY(cudaMemcpyAsync(dA, A, (size_t)M * K, cudaMemcpyHostToDevice, st));
            HOST_TRY(cudaMemcpyAsync(dB, B, (size_t)N * K, cudaMemcpyHostToDevice, st));
        }
        if (bias) HOST_TRY(cudaMemcpyAsync(dbias, bias, (size_t)N * 4, cudaMemcpyHostToDevice, st));
        HOST_TRY(cudaMemcpyAsync(dmult, mult, (size_t)nq * 4, cudaMemcpyHostToDevice, st));
        HOST_TRY(cudaMemcpyAsync(dshift, shift, (size_t)nq * 4, cudaMemcpyHostToDevice, st));
        rc = gemm_i8(dA, K, 1, dB, 1, K, dC, N, bias ? dbias : nullptr, dmult, dshift, per_channel, M, N, K, relu, stream);
        if (rc) return drain(rc);
        HOST_TRY(cudaMemcpyAsync(C, dC, (size_t)M * N, cudaMemcpyDeviceToHost, st));
        HOST_TRY(cudaStreamSynchronize(st));
        return I8_OK;
    }
    cudaEvent_t* ev_in = ctx->ev;            // [i]: chunk i of A (and, for i = 0, B and the vectors) is on the device
    cudaEvent_t* ev_k = ctx->ev + 8;         // [i]: the kernel of chunk i is done
    cudaEvent_t ev_start = ctx->ev[16], ev_done = ctx->ev[17];
    HOST_TRY(cudaEventRecord(ev_start, st)); // the copy streams start after whatever the caller queued on `stream`
    HOST_TRY(cudaStreamWaitEvent(ctx->s_in, ev_start, 0));
    HOST_TRY(cudaStreamWaitEvent(ctx->s_out, ev_start, 0));
    HOST_TRY(cudaMemcpyAsync(dB, B, (size_t)N * K, cudaMemcpyHostToDevice, ctx->s_in));
    if (bias) HOST_TRY(cudaMemcpyAsync(dbias, bias, (size_t)N * 4, cudaMemcpyHostToDevice, ctx->s_in));
    HOST_TRY(cudaMemcpyAsync(dmult, mult, (size_t)nq * 4, cudaMemcpyHostToDevice, ctx->s_in));
    HOST_TRY(cudaMemcpyAsync(dshift, shift, (size_t)nq * 4, cudaMemcpyHostToDevice, ctx->s_in));
    const int rows_per = (((M + nchunks - 1) / nchunks) + 255) / 256 * 256;
    for (int i = 0; i < nchunks; i++) {
        const int r0 = i * rows_per;
        if (r0 >= M) break;
        const int rows = M - r0 < rows_per ? M - r0 : rows_per;
        HOST_TRY(cudaMemcpyAsync(dA + (size_t)r0 * K, A + (size_t)r0 * K, (size_t)rows * K, cudaMemcpyHostToDevice, ctx->s_in));
        HOST_TRY(cudaEventRecord(ev_in[i], ctx->s_in));
        HOST_TRY(cudaStreamWaitEvent(st, ev_in[i], 0));
        rc = gemm_i8(dA + (size_t)r0 * K, K, 1, dB, 1, K, dC + (size_t)r0 * N, N, bias ? dbias : nullptr, dmult, dshift, per_channel,
                     rows, N, K, relu, stream);
        if (rc) return drain(rc);
        HOST_TRY(cudaEventRecord(ev_k[i], st));
        HOST_TRY(cudaStreamWaitEvent(ctx->s_out, ev_k[i], 0));
        HOST_TRY(cudaMemcpyAsync(C + (size_t)r0 * N, dC + (size_t)r0 * N, (size_t)rows * N, cudaMemcpyDeviceToHost, ctx->s_out));
    }
    HOST_TRY(cudaEventRecord(ev_done, ctx->s_out));
    HOST_TRY(cudaStreamWaitEvent(st, ev_done, 0));
    HOST_TRY(cudaStreamSynchronize(st));
#undef HOST_TRY
    return I8_OK;
}

const char* i8_status_string(int status) {
    switch (status) {
        case I8_OK: return "ok";
        case I8_ERR_NULL: return "null pointer";
        case I8_ERR_SHAPE: return "bad shape";
        case I8_ERR_STRIDE: return "bad stride";
        case I8_ERR_ALIGN: return "bad alignment";
        case I8_ERR_RANGE: return "value out of range";
        case I8_ERR_UNSUPPORTED: return "unsupported";
        case I8_ERR_CUDA: return "CUDA call failed";
        case I8_ERR_TIMEOUT: return "a bounded wait expired inside a kernel";
        case I8_ERR_WORKSPACE: return "problem larger than the fixed workspace of the allocation-free variant";
        default: return "unknown status";
    }
}

int i8ops_last_device_status(void* stream) {
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    unsigned v = 0;
    CUDA_TRY(cudaMemcpy(&v, ctx->dev_status, sizeof(v), cudaMemcpyDeviceToHost));
    if (v != 0) {
        const unsigned zero = 0;
        CUDA_TRY(cudaMemcpy(ctx->dev_status, &zero, sizeof(zero), cudaMemcpyHostToDevice));
        return I8_ERR_TIMEOUT;
    }
    return I8_OK;
}

int i8ops_selftest_bounded_wait(int limit_ms, void* stream) {
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    if (limit_ms < 1) limit_ms = 1;
    if (limit_ms > 1000) limit_ms = 1000;
    bounded_wait_selftest_kernel<<<1, 64, 0, (cudaStream_t)stream>>>((long long)limit_ms * 2000000ll, ctx->dev_status);
    CUDA_TRY(cudaGetLastError());
    return I8_OK;
}

int mpc_forward_f32(const float* Adyn, const float* Bdyn, const float* Kinf, const float* x0, const float* d, float* u,
                    float* xs, int batch, int nhorizon, void* stream) {
    t_last_path = I8_PATH_NONE;
    if (batch < 0 || nhorizon < 0) return I8_ERR_SHAPE;
    if (batch == 0 || nhorizon == 0) return I8_OK;
    if (!Adyn || !Bdyn || !Kinf || !x0 || !d || !u) return I8_ERR_NULL;
    if (!aligned16(x0) || !aligned16(d) || !aligned16(u) || (xs && !aligned16(xs))) return I8_ERR_ALIGN;
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    MpcMatrices m;
    for (int r = 0; r < MPC_NX; r++) {
        for (int c = 0; c < MPC_NX; c++) m.At[c][r] = Adyn[r * MPC_NX + c];
        for (int c = 0; c < MPC_NU; c++) m.Bt[c][r] = Bdyn[r * MPC_NU + c];
    }
    for (int r = 0; r < MPC_NU; r++)
        for (int c = 0; c < MPC_NX; c++) m.Kt[c][r] = -Kinf[r * MPC_NX + c];
    cudaStream_t st = (cudaStream_t)stream;
    if (!xs && g_mpc_stream && (int64_t)batch * nhorizon < (1ll << 27)) {
        // streaming kernel: chunks of 256 instances (128 for longer horizons) while two ring slots fit in 72 KB; beyond
        // that the direct kernel
        const int64_t per_inst = MPC_NX * 4 + 16 * (int64_t)nhorizon, tail = MPC_MAX_STAGES * 8 + 16, budget = 72 * 1024;
        const int stages = g_mpc_stream >= 2 && g_mpc_stream <= MPC_MAX_STAGES ? g_mpc_stream : 2;
        const int chunk = stages * 256 * per_inst + tail <= budget ? 256 : (stages * 128 * per_inst + tail <= budget ? 128 : 0);
        if (chunk) {
            const int smem = (int)(stages * chunk * per_inst + tail);
            auto kern = chunk == 256 ? mpc_forward_stream_kernel<256> : mpc_forward_stream_kernel<128>;
            const int slot = chunk == 256 ? 25 : 26;
            if (!ctx->attr_set[slot]) {
                CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)budget));
                ctx->attr_set[slot] = true;
            }
            static thread_local int occ_key = -1, occ_val = 0;    // resident CTAs per SM for (chunk, shared memory)
            if (occ_key != chunk * 1000003 + smem) {
                CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_val, kern, chunk, smem));
                occ_key = chunk * 1000003 + smem;
            }
            const int64_t chunks = ((int64_t)batch + chunk - 1) / chunk;
            // Measured optimum: 384-512 resident threads per SM (2^20 instances, horizon 5: 57 / 45.4 / 53 us with one / two /
            // three CTAs of 256 threads, 57 / 46.5 / 49 / 56 us with two / three / four / six CTAs of 128): fewer leave the
            // fp32 pipe's latency exposed, more slow the memory side down.
            const int want = chunk == 256 ? 2 : 3;
            const int per_sm = occ_val < 1 ? 1 : (occ_val < want ? occ_val : want);
            int64_t blocks = (int64_t)ctx->sm_count * per_sm;
            if (blocks > chunks) blocks = chunks;
            MpcStreamParams sp{x0, d, u, batch, nhorizon, stages, (long long)(g_wait_limit_ns * 2), ctx->dev_status};
            kern<<<(int)blocks, chunk, smem, st>>>(m, sp);
            CUDA_TRY(cudaGetLastError());
            t_last_path = I8_PATH_GENERIC;
            return I8_OK;
        }
    }
    int blocks = (batch + 127) / 128;
    if (blocks > ctx->sm_count * 16) blocks = ctx->sm_count * 16;
    mpc_forward_f32_kernel<<<blocks, 128, 0, st>>>(m, (const float4*)x0, (const float4*)d, (float4*)u, (float4*)xs, batch, nhorizon);
    CUDA_TRY(cudaGetLastError());
    t_last_path = I8_PATH_GENERIC;
    return I8_OK;
}

int i8ops_plan_gemm(int M, int N, int K, int sm_count, i8_plan* out) {
    if (!out) return I8_ERR_NULL;
    if (M <= 0 || N <= 0 || K <= 0 || sm_count <= 0) return I8_ERR_SHAPE;
    const KLoop kl = gemm_kloop(K);
    if (swap_wanted(false, M, N, K, kl.num_kblocks, kl.num_iters, kl.num_kblocks, BK, sm_count)) {
        const SwapPlan sp = plan_swap_auto(M, N, kl.num_iters, sm_count);
        if (sp.pw && sp.stages >= 2) { fill_plan_swap(sp, M, N, out); return I8_OK; }
    }
    fill_plan(plan_tc(false, M, N, K, kl.num_kblocks, kl.num_iters, kl.num_kblocks, BK, sm_count), out);
    return I8_OK;
}

int i8ops_last_plan(i8_plan* out) {
    if (!out) return I8_ERR_NULL;
    *out = t_last_plan;
    return I8_OK;
}

int i8ops_set_class_plan(int shape_cls, int base_m, int base_n, int base_k, int tile_n, int cta_group, int raster_group, int sticky) {
    if (shape_cls < 0 || shape_cls > 2) return I8_ERR_RANGE;
    if (tile_n != 0 && tile_n != 64 && tile_n != 128 && tile_n != 256) return I8_ERR_RANGE;
    if (cta_group < 0 || cta_group > 2 || raster_group < 0 || raster_group > 64 || sticky < -1 || sticky > 1) return I8_ERR_RANGE;
    if (base_m < 0 || base_n < 0 || base_k < 0 || ((base_m == 0) != (base_n == 0)) || ((base_m == 0) != (base_k == 0))) return I8_ERR_RANGE;
    if (cta_group == 2 && tile_n != 0 && tile_n != 256) return I8_ERR_RANGE;      // the pair kernel for GEMMs is 256 wide
    ClassPlan e = {1, base_m, base_n, base_k, tile_n, cta_group, raster_group, sticky};
    if (tile_n == 0 && cta_group == 0 && raster_group == 0 && sticky == -1) e.valid = 0;   // nothing recorded: forget the entry
    g_class_plan[shape_cls] = e;
    return I8_OK;
}

int i8ops_set_class_tile(int shape_cls, int tile_n) {
    return i8ops_set_class_plan(shape_cls, 0, 0, 0, tile_n, 0, 0, -1);
}

int i8ops_tmap_cache_stats(uint64_t* hits, uint64_t* misses) {
    if (!hits || !misses) return I8_ERR_NULL;
    *hits = t_tmap_hits;
    *misses = t_tmap_misses;
    return I8_OK;
}

int i8ops_probe_mma_rate(int tile_n, int reps, int ctas, unsigned long long* out, void* stream) {
    if (!out) return I8_ERR_NULL;
    if (tile_n < 16 || tile_n > 256 || tile_n % 16 != 0 || reps < 64 || reps % 64 != 0 || reps > (1 << 24) || ctas < 1) return I8_ERR_RANGE;
    DeviceCtx* ctx = nullptr;
    int rc = get_ctx(&ctx);
    if (rc) return rc;
    if (ctas > ctx->sm_count) return I8_ERR_RANGE;            // one CTA per SM: more would share tensor cores
    if (!ctx->attr_set[20]) {
        CUDA_TRY(cudaFuncSetAttribute(mma_issue_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PROBE_SMEM));
        ctx->attr_set[20] = true;
    }
    MmaProbeParams p;
    p.n = tile_n; p.reps = reps; p.out = out;
    p.wait_limit_cycles = (long long)(g_wait_limit_ns * 2);
    p.dev_status = ctx->dev_status;
    mma_issue_probe_kernel<<<ctas, PROBE_THREADS, PROBE_SMEM, (cudaStream_t)stream>>>(p);
    CUDA_TRY(cudaGetLastError());
    return I8_OK;
}

int i8ops_last_cuda_error(void) { return t_last_cuda; }
int i8ops_last_path(void) { return t_last_path; }

int i8ops_set_path(int mode) {
    const int prev = g_path_mode;
    if (mode >= 0 && mode <= 6) g_path_mode = mode;
    return prev;
}

void i8ops_set_wait_limit_ms(int ms) {
    if (ms < 1) ms = 1;
    g_wait_limit_ns = (uint64_t)ms * 1000ull * 1000ull;
}

int i8ops_version(void) { return 2; }

}  // extern "C"

// ================================================================================================ allocation-free variant
// gemm_i8_host for callers that must not allocate device memory: the device copies of the operands, of the
// epilogue vectors and of the result live in one array that is part of the library's device image, so the
// driver reserves it on every GPU that loads the library and it stays reserved until the process exits.
namespace i8 {

static __device__ __align__(256) unsigned char g_noalloc_ws[I8OPS_NOALLOC_MAX_BYTES];

// In host code `g_noalloc_ws` is only a handle for the runtime, not an address a kernel or a copy may use; the
// device address is looked up once per device and kept here.
static unsigned char* g_noalloc_ptr[MAX_DEVICES] = {};

static int noalloc_base(unsigned char** out) {
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return cuda_fail(cudaErrorInvalidDevice);
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_noalloc_ptr[dev]) {
        unsigned char* ptr = nullptr;
        CUDA_TRY(cudaGetSymbolAddress((void**)&ptr, g_noalloc_ws));    // the current device's copy of the array
        if (!ptr) return cuda_fail(cudaErrorInvalidSymbol);
        g_noalloc_ptr[dev] = ptr;
    }
    *out = g_noalloc_ptr[dev];
    return I8_OK;
}

}  // namespace i8

extern "C" int gemm_i8_host_noalloc(const int8_t* A, const int8_t* B, int8_t* C, const int32_t* bias, const int32_t* mult,
                                    const int32_t* shift, int per_channel, int M, int N, int K, int relu, void* stream) {
    t_last_path = I8_PATH_NONE;
    if (M < 0 || N < 0 || K < 0) return I8_ERR_SHAPE;
    if (K > 65536) return I8_ERR_RANGE;
    if (M == 0 || N == 0) return I8_OK;
    if (!C || !mult || !shift || (K > 0 && (!A || !B))) return I8_ERR_NULL;
    const int nq = per_channel ? N : 1;
    for (int i = 0; i < nq; i++)
        if (shift[i] < 0 || shift[i] > 31) return I8_ERR_RANGE;
    // every region starts on a 256-byte boundary of the array (the tensor path wants 16-byte aligned operands)
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t szA = up((size_t)M * K), szB = up((size_t)N * K), szC = up((size_t)M * N), szV = up((size_t)N * 4);
    if (szA + szB + szC + 3 * szV > (size_t)I8OPS_NOALLOC_MAX_BYTES) return I8_ERR_WORKSPACE;
    unsigned char* base = nullptr;
    int rc = noalloc_base(&base);
    if (rc) return rc;
    int8_t* dA = (int8_t*)base;
    int8_t* dB = (int8_t*)(base + szA);
    int8_t* dC = (int8_t*)(base + szA + szB);
    int32_t* dbias = (int32_t*)(base + szA + szB + szC);
    int32_t* dmult = (int32_t*)((unsigned char*)dbias + szV);
    int32_t* dshift = (int32_t*)((unsigned char*)dmult + szV);
    // Nothing in the array has to start at zero: every byte the kernel reads below is written by these copies first,
    // and the kernel writes every element of dC that is copied back.  What earlier calls left elsewhere is never read.
    cudaStream_t st = (cudaStream_t)stream;
    if (K > 0) {
        CUDA_TRY(cudaMemcpyAsync(dA, A, (size_t)M * K, cudaMemcpyHostToDevice, st));
        CUDA_TRY(cudaMemcpyAsync(dB, B, (size_t)N * K, cudaMemcpyHostToDevice, st));
    }
    if (bias) CUDA_TRY(cudaMemcpyAsync(dbias, bias, (size_t)N * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(dmult, mult, (size_t)nq * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(dshift, shift, (size_t)nq * 4, cudaMemcpyHostToDevice, st));
    rc = gemm_i8(dA, K, 1, dB, 1, K, dC, N, bias ? dbias : nullptr, dmult, dshift, per_channel, M, N, K, relu, stream);
    if (rc) return rc;
    CUDA_TRY(cudaMemcpyAsync(C, dC, (size_t)M * N, cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    return I8_OK;
}
