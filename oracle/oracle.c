/*
 * CPU oracle for the int8 GEMM / conv2d / batched-GEMM path.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition of what the library computes.  It is linked by the
 * test-suite, by the smoke check and by the benchmark's CPU-baseline leg and by nothing else;
 * it shares no code, header, table or helper with the CUDA path.
 *
 * What is computed, and where the paper defines it:
 *
 *   acc[m][n] = sum_k A[m][k] * B[k][n]      the CPU loop nest of the paper's figure that sets
 *                                            CPU code beside accelerator code for matrix
 *                                            multiplication (Background); operands are 8-bit
 *                                            integers accumulated in 32 bits (Evaluation,
 *                                            "Gemmini Evaluation").
 *   acc      += bias[n]                      Gemmini ISA description (Prompts appendix): with a
 *                                            bias the array computes A*B + bias.
 *   acc       = max(acc, 0) if relu          RELU is one of the activation choices of the same
 *                                            ISA description's execute configuration.
 *   out       = narrow(scale(acc))           reading the accumulator with address bit 29 clear
 *                                            returns scaled-down input-type data with the
 *                                            activation applied (ISA description, continued).
 *
 * The paper shows the scale only as a float argument of its load/store configuration and prints no
 * formula.  The reading taken here is fixed point and exact:
 *     u   = floor( (acc * mult + r) / 2^shift ),  r = 2^(shift-1) for shift >= 1, r = 0 for shift = 0
 *     out = min(127, max(-128, u))
 * evaluated in 64-bit integers, in the order bias, ReLU, scale, clamp.  With mult = 1, shift = 0, no
 * bias and no ReLU this is the saturating C = A*B of the paper's printed Gemmini GEMM listing
 * (NO_ACTIVATION, scale 1.0).
 *
 * The convolution is the direct seven-loop cross-correlation over NHWC activations and KRSC
 * weights (the paper's convolution benchmarks are ResNet-50 layers, "Convolution" subsection); no
 * im2col buffer is formed.  Taps that fall outside the image contribute zero.
 *
 * Accumulation is done in int64 so the oracle itself can never wrap; *overflow is set to 1 when any
 * pre-scale value (after the bias add) leaves the int32 range, which puts the case outside the
 * library's contract.
 *
 * Float-scale read-out (oracle_requant_fscale, oracle_gemm_i8_fscale): the paper's Gemmini listings pass
 * the read-out scale as a single-precision float (the store configuration of the ISA description, e.g. 1.0f in
 * the printed GEMM).  The paper gives no rounding rule; the reading taken here is IEEE-754 binary32 arithmetic, the
 * precision the paper fixes for that argument:
 *     y   = fl32( fl32(t) * scale )      t = acc + bias after the optional ReLU, converted and multiplied with
 *                                        round-to-nearest-even
 *     out = min(127, max(-128, rne(y)))  rne = round to nearest integer, ties to even
 * With scale = 1.0f this is again the saturating C = A*B of the printed listing.
 *
 * Threads (OpenMP) split output rows only; every output element is still produced by the plain
 * loops below in k order.
 */
#include <stdint.h>
#include <stddef.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* floor(x / 2^s) for 0 <= s <= 62 without relying on >> of negative values. */
static int64_t floor_div_pow2(int64_t x, int s)
{
    int64_t d = (int64_t)1 << s;
    int64_t q = x / d;          /* C division truncates toward zero */
    int64_t rem = x % d;
    if (rem < 0) q -= 1;        /* move to the floor for negative non-multiples */
    return q;
}

/* One epilogue: bias -> ReLU -> fixed-point scale with round-half-up -> clamp to int8. */
int32_t oracle_requant(int64_t acc, int32_t bias, int relu, int32_t mult, int32_t shift, int *overflow)
{
    int64_t t = acc + (int64_t)bias;
    if (overflow && (t > (int64_t)INT32_MAX || t < (int64_t)INT32_MIN)) *overflow = 1;
    if (relu && t < 0) t = 0;
    int64_t r = (shift >= 1) ? ((int64_t)1 << (shift - 1)) : 0;
    int64_t u = floor_div_pow2(t * (int64_t)mult + r, shift);
    if (u > 127) u = 127;
    if (u < -128) u = -128;
    return (int32_t)u;
}

/* One float-scale read-out: bias -> ReLU -> binary32 multiply -> round to nearest even -> clamp to int8.
 * (The default rounding mode is round-to-nearest-even; nothing in this library changes it.) */
int32_t oracle_requant_fscale(int64_t acc, int32_t bias, int relu, float scale, int *overflow)
{
    int64_t t = acc + (int64_t)bias;
    if (overflow && (t > (int64_t)INT32_MAX || t < (int64_t)INT32_MIN)) *overflow = 1;
    if (relu && t < 0) t = 0;
    volatile float tf = (float)(int32_t)t;      /* int32 -> binary32, one rounding */
    volatile float y = tf * scale;              /* one binary32 multiplication, one rounding */
    if (y != y) return 0;                       /* NaN scale: defined as 0 */
    if (y >= 127.0f) return 127;
    if (y <= -128.0f) return -128;
    return (int32_t)lrintf(y);                  /* nearest integer, ties to even */
}

/* C[m*ldc+n] = float-scale read-out of sum_k A[..]*B[..]; scale has one entry or N entries. */
int oracle_gemm_i8_fscale(const int8_t *A, int64_t a_rs, int64_t a_cs,
                          const int8_t *B, int64_t b_rs, int64_t b_cs,
                          int8_t *C, int64_t ldc,
                          const int32_t *bias, const float *scale, int per_channel,
                          int M, int N, int K, int relu)
{
    int overflow = 0;
    #pragma omp parallel for schedule(static) reduction(|:overflow)
    for (int m = 0; m < M; m++)
        for (int n = 0; n < N; n++) {
            int64_t acc = 0;
            for (int k = 0; k < K; k++)
                acc += (int32_t)A[m * a_rs + k * a_cs] * (int32_t)B[k * b_rs + n * b_cs];
            int ovf = 0;
            C[m * ldc + n] = (int8_t)oracle_requant_fscale(acc, bias ? bias[n] : 0, relu,
                                                           scale[per_channel ? n : 0], &ovf);
            overflow |= ovf;
        }
    return overflow;
}

/* Raw accumulators of a GEMM (no epilogue), for tests that pin the sum on its own. */
void oracle_gemm_acc(const int8_t *A, int64_t a_rs, int64_t a_cs,
                     const int8_t *B, int64_t b_rs, int64_t b_cs,
                     int64_t *ACC, int M, int N, int K)
{
    #pragma omp parallel for schedule(static)
    for (int m = 0; m < M; m++)
        for (int n = 0; n < N; n++) {
            int64_t acc = 0;
            for (int k = 0; k < K; k++)
                acc += (int32_t)A[m * a_rs + k * a_cs] * (int32_t)B[k * b_rs + n * b_cs];
            ACC[(int64_t)m * N + n] = acc;
        }
}

/* C[m*ldc+n] = epilogue( sum_k A[m*a_rs+k*a_cs] * B[k*b_rs+n*b_cs] ).  All pointers are host memory.
 * bias may be NULL (zero).  mult/shift have one entry (per_channel == 0) or N entries. */
int oracle_gemm_i8(const int8_t *A, int64_t a_rs, int64_t a_cs,
                   const int8_t *B, int64_t b_rs, int64_t b_cs,
                   int8_t *C, int64_t ldc,
                   const int32_t *bias, const int32_t *mult, const int32_t *shift, int per_channel,
                   int M, int N, int K, int relu)
{
    int overflow = 0;
    #pragma omp parallel for schedule(static) reduction(|:overflow)
    for (int m = 0; m < M; m++)
        for (int n = 0; n < N; n++) {
            int64_t acc = 0;
            for (int k = 0; k < K; k++)
                acc += (int32_t)A[m * a_rs + k * a_cs] * (int32_t)B[k * b_rs + n * b_cs];
            int ovf = 0;
            C[m * ldc + n] = (int8_t)oracle_requant(acc, bias ? bias[n] : 0, relu,
                                                    mult[per_channel ? n : 0],
                                                    shift[per_channel ? n : 0], &ovf);
            overflow |= ovf;
        }
    return overflow;
}

/* batch independent GEMMs; problem b uses A + b*a_bs, B + b*b_bs, C + b*c_bs, bias + b*bias_bs
 * (bias_bs == 0: one bias shared by all problems).  mult/shift are shared by all problems. */
int oracle_batched_gemm_i8(const int8_t *A, int64_t a_rs, int64_t a_cs, int64_t a_bs,
                           const int8_t *B, int64_t b_rs, int64_t b_cs, int64_t b_bs,
                           int8_t *C, int64_t ldc, int64_t c_bs,
                           const int32_t *bias, int64_t bias_bs,
                           const int32_t *mult, const int32_t *shift, int per_channel,
                           int batch, int M, int N, int K, int relu)
{
    int overflow = 0;
    #pragma omp parallel for schedule(static) reduction(|:overflow)
    for (int b = 0; b < batch; b++) {
        const int8_t *Ab = A + b * a_bs;
        const int8_t *Bb = B + b * b_bs;
        int8_t *Cb = C + b * c_bs;
        const int32_t *biasb = bias ? bias + b * bias_bs : NULL;
        for (int m = 0; m < M; m++)
            for (int n = 0; n < N; n++) {
                int64_t acc = 0;
                for (int k = 0; k < K; k++)
                    acc += (int32_t)Ab[m * a_rs + k * a_cs] * (int32_t)Bb[k * b_rs + n * b_cs];
                int ovf = 0;
                Cb[m * ldc + n] = (int8_t)oracle_requant(acc, biasb ? biasb[n] : 0, relu,
                                                         mult[per_channel ? n : 0],
                                                         shift[per_channel ? n : 0], &ovf);
                overflow |= ovf;
            }
    }
    return overflow;
}

/* Direct convolution (cross-correlation, no kernel flip), dilation 1, groups 1.
 * x[N][H][W][C], w[K][R][S][C], y[N][P][Q][K];  P = floor((H + 2*pad_h - R)/stride_h) + 1, same for Q.
 * Images n_begin <= n < n_end are computed (a contiguous slab, so a bounded sample can be timed). */
int oracle_conv2d_i8(const int8_t *x, const int8_t *w, int8_t *y,
                     const int32_t *bias, const int32_t *mult, const int32_t *shift, int per_channel,
                     int N, int H, int W, int C, int K, int R, int S,
                     int stride_h, int stride_w, int pad_h, int pad_w, int relu,
                     int n_begin, int n_end)
{
    int P = (H + 2 * pad_h - R) / stride_h + 1;
    int Q = (W + 2 * pad_w - S) / stride_w + 1;
    int overflow = 0;
    (void)N;
    #pragma omp parallel for collapse(2) schedule(static) reduction(|:overflow)
    for (int n = n_begin; n < n_end; n++)
        for (int p = 0; p < P; p++)
            for (int q = 0; q < Q; q++)
                for (int k = 0; k < K; k++) {
                    int64_t acc = 0;
                    for (int r = 0; r < R; r++) {
                        int h = p * stride_h - pad_h + r;
                        if (h < 0 || h >= H) continue;
                        for (int s = 0; s < S; s++) {
                            int ww = q * stride_w - pad_w + s;
                            if (ww < 0 || ww >= W) continue;
                            const int8_t *xp = x + (((int64_t)n * H + h) * W + ww) * C;
                            const int8_t *wp = w + (((int64_t)k * R + r) * S + s) * C;
                            for (int c = 0; c < C; c++)
                                acc += (int32_t)xp[c] * (int32_t)wp[c];
                        }
                    }
                    int ovf = 0;
                    y[(((int64_t)n * P + p) * Q + q) * K + k] =
                        (int8_t)oracle_requant(acc, bias ? bias[k] : 0, relu,
                                               mult[per_channel ? k : 0],
                                               shift[per_channel ? k : 0], &ovf);
                    overflow |= ovf;
                }
    return overflow;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------------------------
 * Fine-grained linear algebra: the forward pass of the TinyMPC primal update that the paper optimises
 * (Code Examples appendix, "TinyMPC Primal Update Forward Pass"; Evaluation, "Fine-Grained Linear Algebra"):
 *     u[i]   = -Kinf * x[i] - d[i]
 *     x[i+1] =  Adyn * x[i] + Bdyn * u[i]            i = 0 .. nhorizon-1
 * Adyn is 12x12, Bdyn 12x4, Kinf 4x12 (row-major), x[0] and d are inputs, u is the output; the last state
 * x[nhorizon] is not needed and not formed.  The paper runs it in fp32 on one instance; here `batch`
 * independent instances share the three matrices.  The oracle evaluates the two equations in double
 * precision, in the plain order written above.  xs (optional, may be NULL) receives x[0..nhorizon-1].
 */
#define MPC_NX 12
#define MPC_NU 4
void oracle_mpc_forward(const double *Adyn, const double *Bdyn, const double *Kinf,
                        const double *x0, const double *d, double *u, double *xs, int batch, int nhorizon)
{
    #pragma omp parallel for schedule(static)
    for (int b = 0; b < batch; b++) {
        double x[MPC_NX], xn[MPC_NX];
        for (int r = 0; r < MPC_NX; r++) x[r] = x0[(int64_t)b * MPC_NX + r];
        for (int i = 0; i < nhorizon; i++) {
            double *ui = u + ((int64_t)b * nhorizon + i) * MPC_NU;
            const double *di = d + ((int64_t)b * nhorizon + i) * MPC_NU;
            if (xs) for (int r = 0; r < MPC_NX; r++) xs[((int64_t)b * nhorizon + i) * MPC_NX + r] = x[r];
            for (int r = 0; r < MPC_NU; r++) {
                double kx = 0.0;
                for (int c = 0; c < MPC_NX; c++) kx += Kinf[r * MPC_NX + c] * x[c];
                ui[r] = -kx - di[r];
            }
            if (i + 1 < nhorizon) {
                for (int r = 0; r < MPC_NX; r++) {
                    double ax = 0.0, bu = 0.0;
                    for (int c = 0; c < MPC_NX; c++) ax += Adyn[r * MPC_NX + c] * x[c];
                    for (int c = 0; c < MPC_NU; c++) bu += Bdyn[r * MPC_NU + c] * ui[c];
                    xn[r] = ax + bu;
                }
                for (int r = 0; r < MPC_NX; r++) x[r] = xn[r];
            }
        }
    }
}
