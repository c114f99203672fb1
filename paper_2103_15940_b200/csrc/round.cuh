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
