// Fused read-out epilogue: bias -> ReLU -> fixed-point scale (round half up) -> saturate to int8.
//
// Two evaluations of the same exact function:
//   requant_wide()  the definition, in 64-bit arithmetic (used by the generic kernel);
//   requant_fast()  the tensor paths' version: per output channel a clamp window [lo, hi] is prepared
//                   once, so that after clamping t = acc + bias into it (a) the saturated result is
//                   unchanged and (b) floor((t*mult + r) / 2^shift) fits in 32 bits, which leaves one
//                   widening multiply-add and one funnel shift per output.
#pragma once
#include <stdint.h>

namespace i8 {

__device__ __forceinline__ int32_t requant_wide(int32_t acc, int32_t bias, int relu, int32_t mult, int32_t shift) {
    long long t = (long long)acc + (long long)bias;
    if (relu && t < 0) t = 0;
    const long long r = shift >= 1 ? (1ll << (shift - 1)) : 0ll;
    long long u = (t * (long long)mult + r) >> shift;   // arithmetic shift on device = floor
    u = u > 127 ? 127 : u;
    u = u < -128 ? -128 : u;
    return (int32_t)u;
}

// Per-output-channel constants of requant_fast.
struct ChanConst {
    int32_t lo, hi;     // clamp window for t = acc + bias (ReLU folded into lo)
    int32_t mult;       // multiplier (canonicalised, see below)
    int32_t shift;      // 0..31
    int32_t rnd;        // 2^(shift-1), or 0 for shift 0
};

// Why the window is exact.  Let b = bit length of |mult| and e = shift + 9 - b.
//   * |t| >= 2^e and mult != 0 imply |t*mult| >= 2^e * 2^(b-1) = 2^(shift+8), so the scaled value is at
//     least 255.5 in magnitude and saturates to the same side as for any larger |t|: clamping t to
//     [-2^e, 2^e] keeps the output.  (mult == 0 gives 0 for every t.)
//   * |t| <= 2^e implies |t*mult + r| < 2^(shift+9) + 2^shift, so the shifted value is below 2^10 in
//     magnitude and its low 32 bits are the value itself.
//   * e >= 31: no clamp is needed; then b <= shift - 22 and |t*mult| < 2^(shift+9) all the same.
//   * e < 0 is raised to 0 (window [-1, 1]): |t| >= 1 still saturates, and |t*mult + r| <= 2^31 + 2^30
//     shifted by shift >= 1 fits; for shift == 0 the value is t*mult itself, which fits unless
//     mult == INT32_MIN and t == -1.  That single pair (mult = -2^31, shift = 0) is replaced by
//     mult = -2^30: every non-zero t saturates to the same side with either multiplier.
__device__ __forceinline__ ChanConst make_chan_const(int32_t mult, int32_t shift, int relu) {
    ChanConst c;
    if (mult == INT32_MIN && shift == 0) mult = -(1 << 30);
    const uint32_t mag = mult < 0 ? (uint32_t)0 - (uint32_t)mult : (uint32_t)mult;
    const int b = 32 - __clz(mag);
    int e = shift + 9 - b;
    if (e < 0) e = 0;
    if (e >= 31) {
        c.lo = INT32_MIN;
        c.hi = INT32_MAX;
    } else {
        c.hi = 1 << e;
        c.lo = -(1 << e);
    }
    if (relu && c.lo < 0) c.lo = 0;
    c.mult = mult;
    c.shift = shift;
    c.rnd = shift >= 1 ? (1 << (shift - 1)) : 0;
    return c;
}

// t = acc + bias already formed by the caller when convenient; this takes acc and bias separately.
__device__ __forceinline__ int32_t requant_fast(int32_t acc, int32_t bias, int32_t lo, int32_t hi, int32_t mult,
                                                int32_t shift, int32_t rnd) {
    int32_t t = acc + bias;
    t = max(t, lo);
    t = min(t, hi);
    const long long p = (long long)t * (long long)mult + (long long)(uint32_t)rnd;
    const uint32_t plo = (uint32_t)p, phi = (uint32_t)((unsigned long long)p >> 32);
    return (int32_t)__funnelshift_r(plo, phi, (uint32_t)shift);   // low word of p >> shift, shift in 0..31
}

// ---------------------------------------------------------------------------------------------------------
// Shift-32 form.  When shift >= 1 and -2^(shift-1) <= mult < 2^(shift-1) (every scale below one half), the
// multiplier can be pre-shifted: m2 = mult * 2^(32-shift) still fits in 32 bits and
//     floor((t*mult + 2^(shift-1)) / 2^shift) = floor((t*m2 + 2^31) / 2^32),
// the same rational number before the floor.  The result is then simply the HIGH word of one 64-bit
// multiply-add, it always fits in 32 bits (|t*m2| <= 2^62), and the saturating pack finishes the clamp;
// no window is needed.  Per output: one add (bias), at most one max (ReLU), one widening multiply-add.
// Per output channel only two words are needed, the bias and m2 (one word when the multiplier is shared).
__device__ __forceinline__ bool make_shift32_mult(int32_t mult, int32_t shift, int32_t& m2) {
    m2 = 0;
    if (shift < 1) return false;
    const int32_t half = 1 << (shift - 1);
    if (mult < -half || mult >= half) return false;
    m2 = (int32_t)((uint32_t)mult << (32 - shift));
    return true;
}

template <bool RELU>
__device__ __forceinline__ int32_t requant_shift32(int32_t acc, int32_t bias, int32_t m2) {
    int32_t t = acc + bias;
    if (RELU) t = max(t, 0);
    const unsigned long long p = (unsigned long long)((long long)t * (long long)m2) + (1ull << 31);
    return (int32_t)(uint32_t)(p >> 32);
}

// Folded shift-32 form.  Because (acc + bias) * m2 + 2^31 = acc * m2 + (bias * m2 + 2^31), the bias can ride in the
// 64-bit addend c = bias * m2 + 2^31 of the one widening multiply-add: |acc * m2| <= 2^62 and |c| <= 2^62 + 2^31, and
// their sum is the in-range value above, so nothing wraps.  ReLU then has to move behind the scale, which is exact
// whenever m2 >= 0: for t = acc + bias < 0 the scaled value floor((t * m2 + 2^31) / 2^32) is <= 0 and becomes 0 either
// way, for t >= 0 it is unchanged.  The saturating pack keeps signs, so that late ReLU is "clear the negative bytes" of
// the packed word (relu_s8x4): two instructions per four outputs instead of one max per output.
__device__ __forceinline__ long long make_fold_addend(int32_t bias, int32_t m2) {
    return (long long)bias * (long long)m2 + (1ll << 31);
}
__device__ __forceinline__ int32_t requant_fold(int32_t acc, int32_t m2, long long c) {
    return (int32_t)(uint32_t)((unsigned long long)((long long)acc * (long long)m2 + c) >> 32);
}
// max(x, 0) on four packed signed bytes: prmt with selector bit 3 set replicates a byte's sign bit over the byte.
__device__ __forceinline__ uint32_t relu_s8x4(uint32_t x) {
    uint32_t neg;
    asm("prmt.b32 %0, %1, %1, 0xba98;" : "=r"(neg) : "r"(x));
    return x & ~neg;
}

// Float-scale read-out (the scale as the single-precision float that the paper's Gemmini listings pass to the store
// configuration): binary32 arithmetic, out = clamp(rne(fl32(fl32(t) * scale))).  The conversion saturates to int32 and
// the caller's saturating pack finishes the clamp; a NaN product converts to 0.
__device__ __forceinline__ int32_t requant_fscale(int32_t acc, int32_t bias, int relu, float scale) {
    int32_t t = acc + bias;
    if (relu) t = max(t, 0);
    return __float2int_rn(__fmul_rn(__int2float_rn(t), scale));
}

// Saturate four 32-bit values to int8 and pack them, v0 in the lowest byte.
// cvt.pack.sat.s8.s32.b32 d, a, b, c  gives  d = (c << 16) | (sat8(a) << 8) | sat8(b).
__device__ __forceinline__ uint32_t pack_sat4(int32_t v0, int32_t v1, int32_t v2, int32_t v3) {
    uint32_t hi, d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(hi) : "r"(v3), "r"(v2), "r"(0));
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(v1), "r"(v0), "r"(hi));
    return d;
}

}  // namespace i8
