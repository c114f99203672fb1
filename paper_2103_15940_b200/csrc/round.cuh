// Device-side rounding to a 1/e/m format and the per-block statistics merge, shared by the
// kernels that round (the rounding pass, the layer-output pass, the FMAC-8 product).
//
// Rounding is roundfp of Section IV-A (nearest representable value, ties to even, denormal range
// kept or flushed); the bins are the stored exponent field of the rounded value with the zero bin
// and the inf/NaN bin split by cause, so that the counters of Section V's statistics (denormal
// fraction, underflow, overflow) need no separate pass.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "qfmt.h"

namespace qfmt {
namespace {

struct QuantParams {
    uint32_t drop;         // 23 - m: mantissa bits removed from a normal value
    uint32_t round_add;    // 2^(drop-1) - 1, or 0 when drop == 0
    uint32_t lsb_mask;     // 1 when drop > 0 (adds the kept LSB: ties go to even)
    uint32_t keep_mask;    // ~(2^drop - 1)
    uint32_t min_normal;   // fp32 bits of 2^E_min
    uint32_t magic;        // fp32 bits of 2^(E_min - m + 23)
    int32_t code_off;      // 127 - bias: fp32 exponent field minus this = stored exponent field
    int32_t top;           // 2^e - 1, the inf/NaN exponent field
    uint32_t keep_denormals;
    float scale;
    uint32_t magic_add;    // ((23 - m) << 23) | 0x400000: exponent field + this = 1.5 * 2^(exponent + 23 - m)
};

// Extra bins after the regular exponent fields 1 .. top-1.
enum : int { kBinZeroIn = 1, kBinRoundedToZero, kBinDenormal, kBinOverflow, kBinInfIn, kBinNanIn, kExtraBins };

__device__ __forceinline__ float add_ieee(float a, float b) {
    float r;
    asm("add.rn.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));  // no .ftz: denormals honoured
    return r;
}
__device__ __forceinline__ float sub_ieee(float a, float b) {
    float r;
    asm("sub.rn.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ float mul_ieee(float a, float b) {
    float r;
    asm("mul.rn.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

// Rounds one element; returns the fp32 container bits and the element's bin.
template <bool kScale>
__device__ __forceinline__ uint32_t quantize_one(uint32_t xb, const QuantParams& p, int& bin) {
    uint32_t yb = kScale ? __float_as_uint(mul_ieee(__uint_as_float(xb), p.scale)) : xb;
    const uint32_t sign = xb & 0x80000000u;  // the scale is positive; a NaN's sign does not survive the multiply
    const uint32_t a = yb & 0x7FFFFFFFu;
    const uint32_t ax = xb & 0x7FFFFFFFu;
    // at or above the smallest normal: round the word itself
    const uint32_t qn = (a + p.round_add + ((a >> p.drop) & p.lsb_mask)) & p.keep_mask;
    // below it: round onto multiples of 2^(E_min-m); cnt is that multiple
    const float magic = __uint_as_float(p.magic);
    const float sum = add_ieee(__uint_as_float(a), magic);
    const uint32_t cnt = __float_as_uint(sum) - p.magic;
    const uint32_t qd = __float_as_uint(sub_ieee(sum, magic));
    uint32_t qa = (a < p.min_normal) ? qd : qn;
    int code = (int)(qa >> 23) - p.code_off;
    bin = code;
    if (code >= p.top) {  // overflow, infinite or NaN
        const bool is_nan = ax > 0x7F800000u;
        qa = is_nan ? 0x7FC00000u : 0x7F800000u;
        bin = p.top + (is_nan ? kBinNanIn : (ax == 0x7F800000u ? kBinInfIn : kBinOverflow));
    } else if (code <= 0) {  // zero or denormal of the format
        bin = p.top + (ax == 0u ? kBinZeroIn : (cnt == 0u ? kBinRoundedToZero : kBinDenormal));
        if (!p.keep_denormals) qa = 0u;
    }
    return sign | qa;
}

// Two elements of binary16 (1/5/10) or bfloat16 (1/8/7) at once: for these two formats the rounding of
// Section IV-A (nearest even onto the format's grid, denormals included, overflow to infinity at
// 2^(E_max+1)) is the IEEE conversion the hardware has, so one packed conversion replaces the integer
// rounding of quantize_one; the classification into bins and the treatment of specials are the same.
// Returns the same containers and bins as quantize_one does, element by element.
template <bool kScale, bool kBf16>
__device__ __forceinline__ void quantize_pair_native(uint32_t xb0, uint32_t xb1, const QuantParams& p, uint32_t& q0,
                                                     uint32_t& q1, int& bin0, int& bin1) {
    constexpr int kM = kBf16 ? 7 : 10;
    constexpr uint32_t kTop = kBf16 ? 255u : 31u;
    const float y0 = kScale ? mul_ieee(__uint_as_float(xb0), p.scale) : __uint_as_float(xb0);
    const float y1 = kScale ? mul_ieee(__uint_as_float(xb1), p.scale) : __uint_as_float(xb1);
    uint32_t pk;  // y1's code in the upper half, y0's in the lower
    if (kBf16) asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(y1), "f"(y0));
    else asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(y1), "f"(y0));
    uint32_t c0, c1;  // containers of the two codes (exact)
    if (kBf16) {
        c0 = pk << 16;
        c1 = pk & 0xFFFF0000u;
    } else {
        float f0, f1;
        asm("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %2; cvt.f32.f16 %0, lo; cvt.f32.f16 %1, hi; }"
            : "=f"(f0), "=f"(f1) : "r"(pk));
        c0 = __float_as_uint(f0);
        c1 = __float_as_uint(f1);
    }
    const uint32_t e0 = (pk >> kM) & kTop, e1 = (pk >> (16 + kM)) & kTop;
    bin0 = (int)e0;
    bin1 = (int)e1;
    if (e0 - 1u >= kTop - 1u) {
        const uint32_t ax = xb0 & 0x7FFFFFFFu, sign = xb0 & 0x80000000u;  // a NaN's sign does not survive the multiply
        if (e0 == kTop) {
            const bool is_nan = ax > 0x7F800000u;
            c0 = sign | (is_nan ? 0x7FC00000u : 0x7F800000u);
            bin0 = p.top + (is_nan ? kBinNanIn : (ax == 0x7F800000u ? kBinInfIn : kBinOverflow));
        } else {
            bin0 = p.top + (ax == 0u ? kBinZeroIn : ((pk & 0x7FFFu) == 0u ? kBinRoundedToZero : kBinDenormal));
            if (!p.keep_denormals) c0 = sign;
        }
    }
    if (e1 - 1u >= kTop - 1u) {
        const uint32_t ax = xb1 & 0x7FFFFFFFu, sign = xb1 & 0x80000000u;
        if (e1 == kTop) {
            const bool is_nan = ax > 0x7F800000u;
            c1 = sign | (is_nan ? 0x7FC00000u : 0x7F800000u);
            bin1 = p.top + (is_nan ? kBinNanIn : (ax == 0x7F800000u ? kBinInfIn : kBinOverflow));
        } else {
            bin1 = p.top + (ax == 0u ? kBinZeroIn : ((pk & 0x7FFF0000u) == 0u ? kBinRoundedToZero : kBinDenormal));
            if (!p.keep_denormals) c1 = sign;
        }
    }
    q0 = c0;
    q1 = c1;
}

// The packed 16-bit codes of two elements of binary16 / bfloat16 by the same conversion: the code of a
// finite result IS the converted half, so only the specials are touched (the library's NaN code, the
// input's sign on it, the flush of denormals).  Same codes and bins as quantize_pack_one.
template <bool kScale, bool kBf16>
__device__ __forceinline__ uint32_t quantize_pack_pair_native(uint32_t xb0, uint32_t xb1, const QuantParams& p, int& bin0,
                                                              int& bin1) {
    constexpr int kM = kBf16 ? 7 : 10;
    constexpr uint32_t kTop = kBf16 ? 255u : 31u;
    const float y0 = kScale ? mul_ieee(__uint_as_float(xb0), p.scale) : __uint_as_float(xb0);
    const float y1 = kScale ? mul_ieee(__uint_as_float(xb1), p.scale) : __uint_as_float(xb1);
    uint32_t pk;  // y1's code in the upper half, y0's in the lower
    if (kBf16) asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(y1), "f"(y0));
    else asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(pk) : "f"(y1), "f"(y0));
    const uint32_t e0 = (pk >> kM) & kTop, e1 = (pk >> (16 + kM)) & kTop;
    bin0 = (int)e0;
    bin1 = (int)e1;
    if (e0 - 1u >= kTop - 1u) {
        const uint32_t ax = xb0 & 0x7FFFFFFFu, sign = (xb0 >> 31) << 15;
        uint32_t c = pk & 0xFFFFu;
        if (e0 == kTop) {
            const bool is_nan = ax > 0x7F800000u;
            c = sign | (kTop << kM) | (is_nan ? (1u << (kM - 1)) : 0u);
            bin0 = p.top + (is_nan ? kBinNanIn : (ax == 0x7F800000u ? kBinInfIn : kBinOverflow));
        } else {
            bin0 = p.top + (ax == 0u ? kBinZeroIn : ((pk & 0x7FFFu) == 0u ? kBinRoundedToZero : kBinDenormal));
            if (!p.keep_denormals) c = sign;
        }
        pk = (pk & 0xFFFF0000u) | c;
    }
    if (e1 - 1u >= kTop - 1u) {
        const uint32_t ax = xb1 & 0x7FFFFFFFu, sign = (xb1 >> 31) << 15;
        uint32_t c = pk >> 16;
        if (e1 == kTop) {
            const bool is_nan = ax > 0x7F800000u;
            c = sign | (kTop << kM) | (is_nan ? (1u << (kM - 1)) : 0u);
            bin1 = p.top + (is_nan ? kBinNanIn : (ax == 0x7F800000u ? kBinInfIn : kBinOverflow));
        } else {
            bin1 = p.top + (ax == 0u ? kBinZeroIn : ((pk & 0x7FFF0000u) == 0u ? kBinRoundedToZero : kBinDenormal));
            if (!p.keep_denormals) c = sign;
        }
        pk = (pk & 0xFFFFu) | (c << 16);
    }
    return pk;
}

// R(S * x) without statistics, for formats with e <= 7: the first rounding of the layer formula.
// The integer pipe runs at half the float pipe's rate, so the rounding is two float operations:
// with C = 1.5 * 2^(max(floor(log2|y|), E_min) + 23 - m) the sum y + C lies in C's binade, whose
// last place is the format's quantum for y; the IEEE addition rounds there to nearest-even (C is
// an even multiple of the quantum) and subtracting C is exact.  Normal and denormal results, both
// signs; a zero result gets y's sign back with an OR.  The exponent is capped at E_max+1 so that C
// stays finite; whatever reaches 2^(E_max+1) becomes infinite.  (A NaN stays some NaN: the addition
// that follows makes it the positive quiet NaN whatever its payload.)
template <bool kScale>
__device__ __forceinline__ uint32_t round_value(uint32_t xb, const QuantParams& p, uint32_t inf_bits) {
    const uint32_t yb = kScale ? __float_as_uint(mul_ieee(__uint_as_float(xb), p.scale)) : xb;
    uint32_t ec = yb & 0x7F800000u;
    ec = ec < p.min_normal ? p.min_normal : ec;
    ec = ec > inf_bits ? inf_bits : ec;
    const float c = __uint_as_float(ec + p.magic_add);
    float q = sub_ieee(add_ieee(__uint_as_float(yb), c), c);
    if (!(fabsf(q) < __uint_as_float(inf_bits)) && q == q) q = copysignf(__uint_as_float(0x7F800000u), q);
    if (!p.keep_denormals && fabsf(q) < __uint_as_float(p.min_normal)) q = 0.0f;
    return __float_as_uint(q) | (yb & 0x80000000u);
}

// Second rounding of the layer formula, with the bin: s is the fp32 sum of two format values
// (e <= 7, so |s| < 2^(E_max+2) and the rounding constant cannot overflow), or inf/NaN.
__device__ __forceinline__ uint32_t round_sum(uint32_t s, const QuantParams& p, int& bin) {
    uint32_t ec = s & 0x7F800000u;
    ec = ec < p.min_normal ? p.min_normal : ec;
    const float c = __uint_as_float(ec + p.magic_add);
    const uint32_t sign = s & 0x80000000u;
    uint32_t q = __float_as_uint(sub_ieee(add_ieee(__uint_as_float(s), c), c)) | sign;
    const uint32_t aq = q & 0x7FFFFFFFu;
    const int code = (int)(aq >> 23) - p.code_off;
    bin = code;
    if ((unsigned)(code - 1) >= (unsigned)(p.top - 1)) {  // not a normal number of the format
        const uint32_t as = s & 0x7FFFFFFFu;
        if (code >= p.top) {
            const bool is_nan = as > 0x7F800000u;
            q = is_nan ? 0x7FC00000u : (sign | 0x7F800000u);
            bin = p.top + (is_nan ? kBinNanIn : (as == 0x7F800000u ? kBinInfIn : kBinOverflow));
        } else {
            bin = p.top + (as == 0u ? kBinZeroIn : (aq == 0u ? kBinRoundedToZero : kBinDenormal));
            if (!p.keep_denormals) q = sign;
        }
    }
    return q;
}

// Rounds one element and returns its packed code, sign | stored exponent | mantissa in the low
// 1 + e + m bits (Definition III.1 with the special encodings of Section III), and the bin.
// For normal results exponent and mantissa fields are the fp32 word's own, re-biased and shifted;
// for denormal results the mantissa is the integer multiple of the smallest denormal that the
// rounding addition leaves in its sum's mantissa field.
template <bool kScale>
__device__ __forceinline__ uint32_t quantize_pack_one(uint32_t xb, const QuantParams& p, int sign_shift, int& bin) {
    uint32_t yb = kScale ? __float_as_uint(mul_ieee(__uint_as_float(xb), p.scale)) : xb;
    const uint32_t sign = (xb >> 31) << sign_shift;
    const uint32_t a = yb & 0x7FFFFFFFu;
    const uint32_t ax = xb & 0x7FFFFFFFu;
    const uint32_t qn = (a + p.round_add + ((a >> p.drop) & p.lsb_mask)) & p.keep_mask;
    const float magic = __uint_as_float(p.magic);
    const float sum = add_ieee(__uint_as_float(a), magic);
    const uint32_t cnt = __float_as_uint(sum) - p.magic;
    const uint32_t qd = __float_as_uint(sub_ieee(sum, magic));
    const uint32_t qa = (a < p.min_normal) ? qd : qn;
    const int code = (int)(qa >> 23) - p.code_off;
    const int m = 23 - (int)p.drop;
    uint32_t packed = (qa - ((uint32_t)p.code_off << 23)) >> p.drop;
    bin = code;
    if (code >= p.top) {  // overflow, infinite or NaN
        const bool is_nan = ax > 0x7F800000u;
        packed = ((uint32_t)p.top << m) | (is_nan ? (1u << (m - 1)) : 0u);
        bin = p.top + (is_nan ? kBinNanIn : (ax == 0x7F800000u ? kBinInfIn : kBinOverflow));
    } else if (code <= 0) {  // zero or denormal of the format
        bin = p.top + (ax == 0u ? kBinZeroIn : (cnt == 0u ? kBinRoundedToZero : kBinDenormal));
        packed = p.keep_denormals ? cnt : 0u;
    }
    return sign | packed;
}

// The same with the denormal grid behind a branch, for tensors in which results below the smallest
// normal are rare (what the paper reports for 1/6/9 and what holds for 1/8/7): the common path is the
// rounding of the word and its re-biased fields only.  If the word's own rounding already reaches a
// normal binade the result is that rounding (for inputs just below 2^E_min both grids give 2^E_min);
// otherwise the input is rounded onto multiples of 2^(E_min-m), and that multiple IS the packed code:
// 2^m, the smallest normal, when the rounding carries.
template <bool kScale>
__device__ __forceinline__ uint32_t quantize_pack_one_rare_denormals(uint32_t xb, const QuantParams& p, int sign_shift,
                                                                     int& bin) {
    const uint32_t yb = kScale ? __float_as_uint(mul_ieee(__uint_as_float(xb), p.scale)) : xb;
    const uint32_t a = yb & 0x7FFFFFFFu;
    const uint32_t qn = (a + p.round_add + ((a >> p.drop) & p.lsb_mask)) & p.keep_mask;
    const int code = (int)(qn >> 23) - p.code_off;
    const int m = 23 - (int)p.drop;
    uint32_t packed = (qn - ((uint32_t)p.code_off << 23)) >> p.drop;
    bin = code;
    if ((unsigned)(code - 1) >= (unsigned)(p.top - 1)) {
        const uint32_t ax = xb & 0x7FFFFFFFu;
        if (code >= p.top) {  // overflow, infinite or NaN
            const bool is_nan = ax > 0x7F800000u;
            packed = ((uint32_t)p.top << m) | (is_nan ? (1u << (m - 1)) : 0u);
            bin = p.top + (is_nan ? kBinNanIn : (ax == 0x7F800000u ? kBinInfIn : kBinOverflow));
        } else {              // below the smallest normal: the denormal grid
            const uint32_t cnt = __float_as_uint(add_ieee(__uint_as_float(a), __uint_as_float(p.magic))) - p.magic;
            if (cnt >> m) {   // carried to 2^E_min
                packed = cnt;
                bin = 1;
            } else {
                bin = p.top + (ax == 0u ? kBinZeroIn : (cnt == 0u ? kBinRoundedToZero : kBinDenormal));
                packed = p.keep_denormals ? cnt : 0u;
            }
        }
    }
    return ((xb >> 31) << sign_shift) | packed;
}

// Packed code of a value that already lies on the format's grid (container bits q as the rounding
// functions return them: finite format values, +-inf, or a NaN).
__device__ __forceinline__ uint32_t encode_container(uint32_t q, const QuantParams& p, int sign_shift) {
    const int m = 23 - (int)p.drop;
    const uint32_t a = q & 0x7FFFFFFFu;
    uint32_t packed;
    if (a >= 0x7F800000u) packed = ((uint32_t)p.top << m) | (a > 0x7F800000u ? (1u << (m - 1)) : 0u);
    else if (a >= p.min_normal) packed = (a - ((uint32_t)p.code_off << 23)) >> p.drop;
    else packed = __float_as_uint(add_ieee(__uint_as_float(a), __uint_as_float(p.magic))) - p.magic;  // multiple of the quantum
    return ((q >> 31) << sign_shift) | packed;
}

// The same when the value's bin is known: bins 1 .. top-1 are the stored exponent fields of normal
// results, which need no case distinction; the sign comes in with one arithmetic shift and a
// bitwise select.
__device__ __forceinline__ uint32_t encode_container(uint32_t q, int bin, const QuantParams& p, int sign_shift) {
    if ((unsigned)(bin - 1) < (unsigned)(p.top - 1)) {
        const uint32_t packed = ((q & 0x7FFFFFFFu) - ((uint32_t)p.code_off << 23)) >> p.drop;
        return packed | ((uint32_t)((int32_t)q >> 31) & (1u << sign_shift));
    }
    return encode_container(q, p, sign_shift);
}

// Packed code of a normal value of the format (container bits q, sign included): subtracting the
// exponent re-bias leaves the sign bit alone, the shift brings exponent and mantissa fields down, and
// the sign is taken from a second shift of the word (bits above the sign position are empty there).
__device__ __forceinline__ uint32_t encode_normal(uint32_t q, const QuantParams& p, int sign_shift) {
    const uint32_t low = (1u << sign_shift) - 1u;
    const uint32_t fields = (q - ((uint32_t)p.code_off << 23)) >> p.drop;
    return (fields & low) | ((q >> (31 - sign_shift)) & ~low);
}

// fp32 container of a packed code.
__device__ __forceinline__ uint32_t unpack_one(uint32_t code, const QuantParams& p, int sign_shift) {
    const int m = 23 - (int)p.drop;
    const uint32_t sign = ((code >> sign_shift) & 1u) << 31;
    const uint32_t E = (code >> m) & (uint32_t)p.top, f = code & ((1u << m) - 1u);
    if (E == (uint32_t)p.top) return sign | (f ? 0x7FC00000u : 0x7F800000u);
    if (E == 0u) {  // f multiples of the smallest denormal 2^(E_min - m): exact, also when that is an fp32 denormal
        const float quantum = mul_ieee(__uint_as_float(p.magic), 1.1920928955078125e-07f);  // magic = 2^(E_min - m + 23)
        return sign | __float_as_uint(mul_ieee((float)f, quantum));
    }
    return sign | ((E + (uint32_t)p.code_off) << 23) | (f << p.drop);
}

// Folds one bin's block total into the device record.
__device__ __forceinline__ void merge_bin(qfmt_stats_t* st, const QuantParams& p, int bin, unsigned long long c) {
    auto add = [](uint64_t* dst, unsigned long long v) { atomicAdd((unsigned long long*)dst, v); };
    if (bin < p.top) {
        add(&st->hist[bin], c);
        return;
    }
    switch (bin - p.top) {
        case kBinZeroIn: add(&st->hist[0], c); add(&st->n_zero_in, c); break;
        case kBinRoundedToZero: add(&st->hist[0], c); add(&st->n_underflow, c); break;
        case kBinDenormal:
            add(&st->hist[0], c); add(&st->n_denormal, c);
            if (!p.keep_denormals) add(&st->n_underflow, c);
            break;
        case kBinOverflow: add(&st->hist[p.top], c); add(&st->n_overflow, c); break;
        case kBinInfIn: add(&st->hist[p.top], c); add(&st->n_inf_in, c); break;
        case kBinNanIn: add(&st->hist[p.top], c); add(&st->n_nan, c); break;
        default: break;
    }
}

inline QuantParams make_params(const qfmt_format_t& f) {
    QuantParams p;
    const int bias = (1 << (f.e - 1)) - 1;
    const int emin = 1 - bias;
    p.drop = 23u - (uint32_t)f.m;
    p.round_add = p.drop ? ((1u << (p.drop - 1)) - 1u) : 0u;
    p.lsb_mask = p.drop ? 1u : 0u;
    p.keep_mask = ~((1u << p.drop) - 1u);
    p.min_normal = (uint32_t)(emin + 127) << 23;
    p.magic = (uint32_t)(emin - f.m + 23 + 127) << 23;
    p.code_off = 127 - bias;
    p.top = (1 << f.e) - 1;
    p.keep_denormals = f.denormals ? 1u : 0u;
    p.scale = f.loss_scale;
    p.magic_add = (p.drop << 23) | 0x00400000u;
    return p;
}

}  // namespace
}  // namespace qfmt
