/*
 * i8ops — int8 GEMM, NHWC conv2d and batched/skinny GEMM for NVIDIA B200 (sm_100a), each with a fused
 * read-out epilogue (int32 bias, optional ReLU, fixed-point scale, saturating narrow to int8).
 *
 * These are the tensor operations that the Autocomp paper (arXiv 2505.18574) optimises on a
 * Gemmini-style accelerator: 8-bit integer operands accumulated in 32 bits (Evaluation, "Gemmini
 * Evaluation"), computed tile by tile as  move-in -> matrix unit -> accumulator -> scaled move-out
 * (Background, the figure that sets CPU code beside accelerator code; Gemmini ISA description in the
 * Prompts appendix).  Here the scratchpad is shared memory fed by TMA, the matrix unit is
 * tcgen05.mma kind::i8, the accumulator is tensor memory, and the move-out is the fused epilogue.
 *
 * Epilogue, applied to every accumulator acc (exact, evaluated in 64-bit integers):
 *     t   = acc + bias[n]                      (bias == NULL means 0; ISA description: C = A*B + bias)
 *     t   = max(t, 0)            if relu       (RELU activation of the ISA's execute configuration)
 *     u   = floor((t * mult[n] + r) / 2^shift[n]),   r = 2^(shift-1) if shift >= 1 else 0
 *     out = min(127, max(-128, u))             (reading the accumulator as scaled-down input-type
 *                                               data, ISA description continued)
 * The paper shows the scale only as a float argument; this library fixes it as the multiplier/shift
 * pair above (round half toward +infinity).  mult = 1, shift = 0, no bias, no ReLU reproduces the
 * saturating C = A*B of the paper's printed Gemmini GEMM listing.
 *
 * Conventions for every compute entry point below
 *   - All tensor, bias, mult and shift pointers are DEVICE pointers owned by the caller (the *_host
 *     variants take HOST pointers and say so).  Inputs are never written.  The output must not
 *     overlap any input.
 *   - Strides are in elements (= bytes for the int8 tensors).
 *   - mult / shift hold one entry (per_channel == 0) or N entries indexed by output channel
 *     (per_channel != 0).  Any int32 multiplier is legal; every shift must lie in [0, 31] (not
 *     checked on the device: the caller guarantees it, the host variants check it).
 *   - Contract on magnitudes: acc + bias must fit in int32 (guaranteed for K <= 65536 with
 *     |bias| < 2^30); behaviour beyond that is unspecified.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = default stream).
 *   - The return value is an i8_status for errors the host can detect before launching; nothing is
 *     launched when it is non-zero.  The library never throws, aborts or exits.
 *   - Every wait inside the kernels is bounded.  If one ever expires the kernel stops early, leaves
 *     the rest of the output unwritten and records the fact; i8ops_last_device_status() reports it.
 */
#ifndef I8OPS_H
#define I8OPS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    I8_OK = 0,
    I8_ERR_NULL = 1,        /* a required pointer is NULL */
    I8_ERR_SHAPE = 2,       /* a negative extent, or a convolution with an empty output */
    I8_ERR_STRIDE = 3,      /* neither stride of an operand is 1, or a leading dimension is too small */
    I8_ERR_ALIGN = 4,       /* reserved: misaligned operands are served by the generic kernel instead */
    I8_ERR_RANGE = 5,       /* K > 65536, or (host variants) a shift outside [0, 31] */
    I8_ERR_UNSUPPORTED = 6, /* stride or padding outside what the convolution supports */
    I8_ERR_CUDA = 7,        /* a CUDA runtime or driver call failed; see i8ops_last_cuda_error() */
    I8_ERR_TIMEOUT = 8,     /* a bounded wait inside a kernel expired (device status only) */
    I8_ERR_WORKSPACE = 9    /* gemm_i8_host_noalloc: the problem does not fit its fixed device workspace */
} i8_status;

/* Which kernel family served the most recent compute call of this thread (for tests and tuning). */
typedef enum {
    I8_PATH_NONE = 0,       /* nothing launched (empty problem or error) */
    I8_PATH_GENERIC = 1,    /* one-thread-per-output kernel: any strides, any alignment */
    I8_PATH_TENSOR = 2,     /* TMA -> shared memory ring -> tcgen05.mma kind::i8 -> tensor memory -> epilogue */
    I8_PATH_SMALL = 3,      /* small-tile tensor path: paired 64x64 problems */
    I8_PATH_TENSOR_2SM = 4, /* tensor path on clusters of two CTAs (tcgen05.mma.cta_group::2, 256 x 256 tiles) */
    I8_PATH_CONV_SLAB = 5,  /* stride-1 convolution with the input slab resident in shared memory and reused across taps */
    I8_PATH_CHANNEL_MAJOR = 6,     /* tensor path computing the transposed product: 128 output channels on the tensor-memory
                                      lanes, a strip of output rows on the columns (strip width chosen per problem) */
    I8_PATH_CHANNEL_MAJOR_2SM = 7  /* the same on clusters of two CTAs: 256 output channels per tile */
} i8_path;

/*
 * C[m*ldc + n] = epilogue( sum_k A[m*a_rs + k*a_cs] * B[k*b_rs + n*b_cs] ),  0 <= m < M, 0 <= n < N.
 * (The product of the paper's matrix-multiplication figure; int8 x int8 accumulated in int32.)
 *   A, B   device, int8.  Exactly one of (a_rs, a_cs) and one of (b_rs, b_cs) must be 1; the other is the
 *          leading dimension (>= the extent it strides over).  Row-major A is (a_rs = lda, a_cs = 1);
 *          column-major B is (b_rs = 1, b_cs = ldb).
 *   C      device, int8, row-major, ldc >= N.
 *   bias   device, int32[N], or NULL.
 *   mult, shift, per_channel, relu   see the epilogue above.
 * The tensor path fetches operands in place when their base addresses and leading dimensions are multiples of 16 bytes
 * (either storage order of either operand).  Other operands are first packed into K-contiguous, zero-padded copies in a
 * workspace that is allocated and released in stream order from a memory pool the library keeps per device (the call
 * stays asynchronous and may be captured into a CUDA graph; make the first such call on a device outside any capture);
 * problems below 2^18 multiply-accumulates, or whose copies would exceed 256 MiB, take the one-thread-per-output kernel
 * instead.  Same results on every path.  i8ops_last_gemm_packed() tells whether the last call packed its operands.
 * Errors: I8_ERR_NULL, I8_ERR_SHAPE (negative M, N or K), I8_ERR_STRIDE, I8_ERR_RANGE, I8_ERR_CUDA.
 * M == 0 or N == 0 returns I8_OK and launches nothing; K == 0 yields epilogue(0).
 */
int gemm_i8(const int8_t* A, int64_t a_rs, int64_t a_cs,
            const int8_t* B, int64_t b_rs, int64_t b_cs,
            int8_t* C, int64_t ldc,
            const int32_t* bias, const int32_t* mult, const int32_t* shift, int per_channel,
            int M, int N, int K, int relu, void* stream);

/*
 * Raw read-out: D[m*ldd + n] (+)= sum_k A[..] * B[..] as int32, with no bias, activation or scale.  This is the
 * accumulator read as accumulator-type data (Gemmini ISA description, continued: address bit 29 set), and with
 * accumulate != 0 the product is added to what D already holds (address bit 30: accumulate instead of overwrite),
 * which lets a caller split K across calls.  D is device int32, row-major, ldd >= N; other arguments as gemm_i8
 * (misaligned operands are packed first, as there).
 * The sums must fit in int32 (always true for a single product with K <= 65536).
 * Errors: I8_ERR_NULL, I8_ERR_SHAPE, I8_ERR_STRIDE, I8_ERR_RANGE, I8_ERR_CUDA.
 */
int gemm_i8_raw(const int8_t* A, int64_t a_rs, int64_t a_cs,
                const int8_t* B, int64_t b_rs, int64_t b_cs,
                int32_t* D, int64_t ldd, int accumulate,
                int M, int N, int K, void* stream);

/*
 * gemm_i8 with the read-out scale given as a single-precision float, as the paper's Gemmini listings pass it (the scale
 * argument of the ISA description's store configuration, 1.0f in the printed GEMM):
 *     t = acc + bias[n];  t = max(t, 0) if relu;  out = min(127, max(-128, rne(fl32(fl32(t) * scale[n]))))
 * fl32 = rounding to IEEE-754 binary32 (nearest, ties to even), applied to the conversion of t and to the product;
 * rne = nearest integer, ties to even (the paper states no rounding rule; this is the reading taken).  A NaN product
 * yields 0.  scale: device, float[1] (per_channel == 0) or float[N].  Other arguments, layouts and errors as gemm_i8
 * (I8_ERR_NULL also for a NULL scale).  K-contiguous aligned operands run on the channel-major tensor kernel in place,
 * other operands through packed copies as in gemm_i8.
 */
int gemm_i8_fscale(const int8_t* A, int64_t a_rs, int64_t a_cs,
                   const int8_t* B, int64_t b_rs, int64_t b_cs,
                   int8_t* C, int64_t ldc,
                   const int32_t* bias, const float* scale, int per_channel,
                   int M, int N, int K, int relu, void* stream);

/*
 * `batch` independent products (the paper's fine-grained linear algebra: many small, low-reuse
 * products, Evaluation "Fine-Grained Linear Algebra"; also its column-dominant GEMM shapes).
 * Problem b uses A + b*a_bs, B + b*b_bs, C + b*c_bs and bias + b*bias_bs (bias_bs == 0: one bias
 * shared by all problems); mult/shift are shared by all problems.  Other arguments as gemm_i8.
 * Kernels: problems up to 64 x 64 x 64 run two to an instruction on the paired small-tile kernel; larger ones with
 * 16-byte aligned slices run in ONE launch of the large-tile kernel whose tile schedule covers all problems (row-major
 * A, either storage order of B, batch strides that are whole rows), else one launch per problem, else the
 * one-thread-per-output kernel.  Same results on every path.
 * Errors as gemm_i8, plus I8_ERR_SHAPE for a negative batch.
 */
int batched_gemm_i8(const int8_t* A, int64_t a_rs, int64_t a_cs, int64_t a_bs,
                    const int8_t* B, int64_t b_rs, int64_t b_cs, int64_t b_bs,
                    int8_t* C, int64_t ldc, int64_t c_bs,
                    const int32_t* bias, int64_t bias_bs,
                    const int32_t* mult, const int32_t* shift, int per_channel,
                    int batch, int M, int N, int K, int relu, void* stream);

/*
 * y[n][p][q][k] = epilogue( sum_{r,s,c} x[n][p*stride_h - pad_h + r][q*stride_w - pad_w + s][c] * w[k][r][s][c] )
 * (the paper's ResNet-50 convolution benchmarks, Evaluation "Convolution", lowered to an implicit GEMM
 * with M = N*P*Q, N = K filters, K = R*S*C).  Cross-correlation (no kernel flip); taps outside the image
 * contribute 0; dilation 1, groups 1.
 *   x  device int8 [N][H][W][C] (NHWC, dense);  w  device int8 [K][R][S][C] (dense);
 *   y  device int8 [N][P][Q][K] (dense),  P = floor((H + 2*pad_h - R)/stride_h) + 1, Q likewise.
 *   bias/mult/shift indexed by filter k.
 * Layers that the implicit-GEMM loads do not take (an activation tensor below 128 KiB, a stride above 8, a filter side or
 * padding above 16, a channel count that is not a multiple of 32, misaligned bases) run as an unfold pass into the GEMM
 * form's A matrix followed by the tensor GEMM; that matrix (N*P*Q rows of R*S*C bytes rounded up to 16, plus a padded
 * copy of the filters when C % 16 != 0; at most 256 MiB together, else the one-thread-per-output kernel serves the call)
 * is allocated and released in stream order from a memory pool the library keeps per device, so the call stays
 * asynchronous and may be captured into a CUDA graph.
 * The first such call on a device creates the pool: make it outside any stream capture.
 * i8ops_last_conv_unfolded() tells whether the most recent convolution of this thread ran that way.
 * Errors: I8_ERR_NULL, I8_ERR_SHAPE (a non-positive extent or an empty output), I8_ERR_UNSUPPORTED
 * (stride < 1, pad < 0), I8_ERR_RANGE (R*S*C > 65536), I8_ERR_CUDA.
 */
int conv2d_i8(const int8_t* x, const int8_t* w, int8_t* y,
              const int32_t* bias, const int32_t* mult, const int32_t* shift, int per_channel,
              int N, int H, int W, int C, int K, int R, int S,
              int stride_h, int stride_w, int pad_h, int pad_w, int relu, void* stream);

int i8ops_last_conv_unfolded(void);
/* Whether the most recent gemm_i8 of this thread ran on packed copies of its operands (see gemm_i8). */
int i8ops_last_gemm_packed(void);

/*
 * Host-buffer variants: every pointer is HOST memory (pinned memory makes the copies asynchronous).
 * The call copies the operands to a device workspace that the library keeps per device (grown with
 * cudaMalloc when a larger problem arrives, never shrunk), runs the same kernels, copies the result
 * back and synchronises `stream` before returning.  Problems with 2048 rows or more are cut into row chunks whose
 * copy-in, kernel and copy-out overlap on three streams (two of them internal).  They also check every shift (I8_ERR_RANGE).
 * Tight layouts only: A row-major [M][K], B column-major (K contiguous, [N][K]), C row-major [M][N].
 * The workspace, the internal streams and their events belong to the device, not to the call: calls on one device are
 * serialised by a lock inside the library (a second host thread waits until the first call has returned), so
 * concurrent callers are safe but gain nothing.  If a CUDA call fails part-way, everything already queued is allowed
 * to finish before the error is returned; C is then unspecified.
 */
int gemm_i8_host(const int8_t* A, const int8_t* B, int8_t* C,
                 const int32_t* bias, const int32_t* mult, const int32_t* shift, int per_channel,
                 int M, int N, int K, int relu, void* stream);

/*
 * gemm_i8_host without any allocation (the paper has no counterpart; this exists for callers, not for the method).
 * Some programs may not allocate device memory once they are running: a control loop with a fixed memory budget
 * (the setting of the paper's TinyMPC benchmark), a plug-in inside a host application that owns the GPU's memory
 * pool, or code that runs while the allocator is off limits because an allocation would synchronise the device.
 * For them this entry point does what gemm_i8_host does, but its device copies of A, B, bias, mult, shift and C
 * live in a fixed array of I8OPS_NOALLOC_MAX_BYTES that is part of the library's device image: every GPU that
 * loads the library sets that much memory aside until the process exits, whether or not this function is called.
 * It calls no cudaMalloc, cudaFree or other allocating routine, creates no streams or events, and does all its
 * copies and its kernel on `stream`, which it synchronises before returning.
 *   Arguments, layouts and results as gemm_i8_host (HOST pointers; tight row-major A and C, K-contiguous B).
 *   Limit: with every region rounded up to 256 bytes, M*K + N*K + M*N + 3 * 4*N must not exceed
 *   I8OPS_NOALLOC_MAX_BYTES (e.g. 2048 x 2048 x 2048 fits, 4096^3 does not); larger problems return
 *   I8_ERR_WORKSPACE and nothing is launched or copied.
 *   The first call on each device looks up the array's device address (with that device current) and may load
 *   kernels; make that first call outside any stream capture.
 *   All calls on a device share the one array.  It keeps whatever the last call left; nothing in it needs
 *   clearing, because each call overwrites every byte it later reads.  Two calls that are in flight on the same
 *   GPU at the same time (from two host threads or processes sharing the context) race on it: serialise them.
 * Errors: as gemm_i8_host, plus I8_ERR_WORKSPACE.
 */
#define I8OPS_NOALLOC_MAX_BYTES (16 * 1024 * 1024)
int gemm_i8_host_noalloc(const int8_t* A, const int8_t* B, int8_t* C,
                         const int32_t* bias, const int32_t* mult, const int32_t* shift, int per_channel,
                         int M, int N, int K, int relu, void* stream);

/* Human-readable name of an i8_status. */
const char* i8_status_string(int status);

/* Synchronises `stream`, then returns I8_OK, I8_ERR_TIMEOUT if a bounded wait expired in any kernel of
 * this library on the current device since the last call, or I8_ERR_CUDA.  Clears the record. */
int i8ops_last_device_status(void* stream);

/*
 * Forward pass of the TinyMPC primal update, the paper's fine-grained linear-algebra benchmark (Code Examples
 * appendix, "TinyMPC Primal Update Forward Pass"), for `batch` independent instances that share the matrices:
 *     u[i] = -Kinf * x[i] - d[i];   x[i+1] = Adyn * x[i] + Bdyn * u[i];   i = 0 .. nhorizon-1  (x[nhorizon] is not formed)
 *   Adyn [12][12], Bdyn [12][4], Kinf [4][12]   HOST pointers, row-major fp32 (copied into the launch's arguments)
 *   x0 [batch][12], d [batch][nhorizon][4]      device, fp32, 16-byte aligned
 *   u  [batch][nhorizon][4]                     device output, fp32, 16-byte aligned
 *   xs [batch][nhorizon][12] or NULL            device output: the states x[0..nhorizon-1]
 * Arithmetic is fp32 with fused multiply-adds in ascending index order (the paper's precision; two output rows share
 * one packed instruction, each half rounded as the scalar instruction would).
 * Without xs and for horizons up to 12 steps, persistent CTAs stream chunks of 128 instances through a shared-memory ring
 * (bulk copies in, bulk copies out; every wait bounded, see i8ops_last_device_status); otherwise one thread per
 * instance loads and stores its own records.  Same arithmetic, same results.
 * Errors: I8_ERR_SHAPE (negative batch or nhorizon), I8_ERR_NULL, I8_ERR_ALIGN, I8_ERR_CUDA.
 */
int mpc_forward_f32(const float* Adyn, const float* Bdyn, const float* Kinf, const float* x0, const float* d, float* u,
                    float* xs, int batch, int nhorizon, void* stream);

/* Tile plan of gemm_i8's tensor path for one shape, and its reuse across shapes of the same aspect class: the
 * analogue of the paper's schedule reuse (section "Improving Sample Efficiency With Schedule Reuse": a schedule found
 * for one GEMM is replayed on GEMMs of the same aspect class: square, column-dominant, row-dominant). */
typedef struct {
    int shape_class;     /* 0 square (neither side 8x the other), 1 column-dominant (M >= 8N), 2 row-dominant (N >= 8M) */
    int tile_m, tile_n;  /* output tile: 128 (one CTA) or 256 (a CTA pair) x {64, 128, 256} */
    int stages;          /* ring slots of 128 bytes of K */
    int cta_group;       /* 1: one CTA per tile; 2: a cluster of two CTAs per tile (tcgen05.mma.cta_group::2) */
    int raster_group;    /* block rows walked through all block columns before moving on (L2 reuse) */
    int sticky;          /* 1: every worker keeps one block column for the whole kernel */
    int m_tiles, n_tiles;
    int workers;         /* CTAs (cta_group 1) or CTA pairs (cta_group 2) launched */
    int waves;           /* ceil(tiles / workers) */
    int b_resident;      /* B fetched once per CTA and kept in shared memory */
    int epilogue_warps;
    int kernel;          /* 0: large-tile kernel (rows of C on the tensor-memory lanes); 1: channel-major kernel: tile_m is
                            then the strip of rows per tile (a multiple of 16) and tile_n the channel block, 128 or 256 */
} i8_plan;

/* Fills *out with the plan gemm_i8 would launch for K-contiguous operands of shape (M, N, K) on a device with sm_count
 * SMs: the launch code and this query call the same planning function.  Host only; no CUDA call.
 * Errors: I8_ERR_NULL, I8_ERR_SHAPE (a non-positive argument). */
int i8ops_plan_gemm(int M, int N, int K, int sm_count, i8_plan* out);

/* The plan of the most recent launch of the large-tile tensor kernel made by this thread (GEMM or convolution). */
int i8ops_last_plan(i8_plan* out);

/* Records a schedule for every later GEMM of class shape_class (the paper's reuse of one shape's schedule on the other
 * shapes of its class), replacing the built-in choice for the fields that are set:
 *   base_m, base_n, base_k   the shape the schedule was found on: the entry then applies to shapes whose M, N and K each
 *                            lie within a factor of four of it; all three 0: the entry applies to the whole class
 *   tile_n        64, 128 or 256; 0 = cost model (a width much wider than the problem is ignored)
 *   cta_group     1 or 2; 0 = measured crossover rule (2 implies 256-wide tiles)
 *   raster_group  1..64; 0 = default (16)
 *   sticky        1 = column-sticky order where it is legal, 0 = never, -1 = rule
 * All fields at "no choice" forgets the entry.  The library starts with two entries, seeded from its tuned plans for
 * 8192^3 (square) and 262144 x 64 x 256 (column-dominant).  Not thread-safe against concurrent launches.
 * Errors: I8_ERR_RANGE. */
int i8ops_set_class_plan(int shape_class, int base_m, int base_n, int base_k, int tile_n, int cta_group, int raster_group,
                         int sticky);

/* Shorthand: record only a tile width for the whole class (tile_n == 0 forgets the class entry). */
int i8ops_set_class_tile(int shape_class, int tile_n);

/* Tensor maps are cached per host thread, keyed on base address and geometry.  Reports this thread's cache hits and
 * misses so far (for tests and tuning).  Errors: I8_ERR_NULL. */
int i8ops_tmap_cache_stats(uint64_t* hits, uint64_t* misses);

/* Measures the issue rate of the tensor-core instruction every int8 kernel here is built on (no counterpart in the
 * paper; it gives the roofline its measured int8 denominator).  `ctas` CTAs, one per SM, each issue `reps`
 * tcgen05.mma kind::i8 instructions of 128 x tile_n x 32 on operands that already sit in shared memory and wait for
 * the last to finish.  Asynchronous on `stream`.
 *   out   device, uint64 [ctas][4], written by the kernel: SM cycles spent issuing; SM cycles until the last
 *         instruction completed; nanoseconds (global timer) until then; the SM's id.  A CTA whose bounded wait expired
 *         writes 0 for the second and third value.
 *   Peak of the chip = ctas * reps * 2 * 128 * tile_n * 32 operations / the largest of the nanosecond figures.
 * Errors: I8_ERR_NULL, I8_ERR_RANGE (tile_n not a multiple of 16 in 16..256, reps not a multiple of 64 in 64..2^24,
 * ctas outside 1..SM count), I8_ERR_CUDA. */
int i8ops_probe_mma_rate(int tile_n, int reps, int ctas, unsigned long long* out, void* stream);

/* Self-test of the failure path (no counterpart in the paper): launches one small CTA that waits, for at most
 * `limit_ms` (1..1000) milliseconds, on a barrier that nothing signals.  The kernel returns by itself and the next
 * i8ops_last_device_status() reports I8_ERR_TIMEOUT.  Nothing faults, traps or hangs. */
int i8ops_selftest_bounded_wait(int limit_ms, void* stream);

/* cudaError_t of the most recent failed CUDA call made by this library on this thread (0 if none). */
int i8ops_last_cuda_error(void);

/* i8_path of the most recent compute call made by this thread. */
int i8ops_last_path(void);

/* Restrict dispatch: 0 = automatic (default), 1 = always the generic kernel, 2 = GEMMs and convolutions take the
 * two-SM tensor kernel whenever the layout allows the tensor path (also where its large tiles do not pay),
 * 3 = automatic among the large-tile kernels only (no slab kernel, no channel-major kernel),
 * 4 = GEMMs and implicit-GEMM convolutions take the channel-major kernel whenever the layout allows the tensor path
 *     (single CTAs or CTA pairs by its cost model), 5 = the same on CTA pairs whenever there are more than 128 channels,
 *     6 = the same on single CTAs only.
 * Returns the previous setting. */
int i8ops_set_path(int mode);

/* Upper limit, in milliseconds, for any single wait inside a kernel (default 2000). */
void i8ops_set_wait_limit_ms(int ms);

/* Library ABI version (bumped when a signature changes). */
int i8ops_version(void);

#ifdef __cplusplus
}
#endif
#endif /* I8OPS_H */
