// Rounding of fp32 tensors to a 1/e/m format with range statistics in the same pass.
//
// The operation is the roundfp kernel of Section IV-A (nearest representable value with e
// exponent bits and m mantissa bits, denormal range allowed or not), preceded by the
// loss-scale multiply of Section II and followed, in registers, by the classification the
// paper's statistics need (Section V: denormal fraction per tensor; the exponent histogram
// gives the width of the range of values).
//
// Design (HBM-bound: 4 bytes read + 4 bytes written per element, a few dozen integer
// instructions in between):
//   * 128-bit streaming loads and stores, several in flight per thread, a grid sized to the
//     SM count so that the per-block merge happens once per block.
//   * Rounding works on the fp32 bit pattern.  Values at or above the format's smallest normal
//     are rounded by an integer add-and-mask on the word (the carry moves into the exponent
//     field by itself).  Values below it are rounded onto the denormal grid by adding
//     2^(E_min-m+23) with an IEEE add (denormals honoured) and reading the integer multiple of
//     the denormal quantum straight out of the sum's mantissa field.
//   * Every element is assigned ONE bin: its stored exponent field, with the zero bin and the
//     inf/NaN bin split by cause (zero input / rounded to zero / denormal; overflow / infinite
//     input / NaN input).  The block keeps a histogram privatised per lane, [bin][lane], so
//     that a warp's 32 shared-memory atomics always hit 32 different banks whatever the data
//     look like.  At the end each bin's 32 lanes are summed with a warp reduction and merged
//     into the 64-bit device record with one atomic per non-empty bin per block; the split
//     bins are folded into hist[0], hist[2^e-1] and the counters there.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

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

__device__ __forceinline__ uint4 load_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void store_stream(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
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

constexpr int kThreads = 512;
constexpr int kUnroll = 4;  // 128-bit loads in flight per thread

// in/out point at the first element; `head` elements precede the 16-byte aligned body of n4
// vectors and `tail` elements follow it.
template <bool kOut, bool kStats, bool kScale>
__global__ void __launch_bounds__(kThreads)
quantize_stats_kernel(const uint32_t* in, uint32_t* out, uint32_t head,
                      unsigned long long n4, uint32_t tail, QuantParams p, qfmt_stats_t* __restrict__ stats,
                      unsigned long long n_total) {
    extern __shared__ uint32_t lane_hist[];  // [(top + kExtraBins)][32]
    const int nbins = p.top + kExtraBins;
    const int lane = threadIdx.x & 31;
    if (kStats) {
        for (int i = threadIdx.x; i < nbins * 32; i += kThreads) lane_hist[i] = 0u;
        __syncthreads();
    }
    const uint4* in4 = reinterpret_cast<const uint4*>(in + head);
    uint4* out4 = reinterpret_cast<uint4*>(out + head);

    const unsigned long long stride = (unsigned long long)gridDim.x * (kThreads * kUnroll);
    for (unsigned long long base = (unsigned long long)blockIdx.x * (kThreads * kUnroll); base < n4; base += stride) {
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kThreads + threadIdx.x;
            if (idx < n4) v[u] = load_stream(in4 + idx);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kThreads + threadIdx.x;
            if (idx < n4) {
                int b0, b1, b2, b3;
                uint4 q;
                q.x = quantize_one<kScale>(v[u].x, p, b0);
                q.y = quantize_one<kScale>(v[u].y, p, b1);
                q.z = quantize_one<kScale>(v[u].z, p, b2);
                q.w = quantize_one<kScale>(v[u].w, p, b3);
                if (kOut) store_stream(out4 + idx, q);
                if (kStats) {
                    atomicAdd(&lane_hist[b0 * 32 + lane], 1u);
                    atomicAdd(&lane_hist[b1 * 32 + lane], 1u);
                    atomicAdd(&lane_hist[b2 * 32 + lane], 1u);
                    atomicAdd(&lane_hist[b3 * 32 + lane], 1u);
                }
            }
        }
    }
    // unaligned head and tail (at most 3 elements each), block 0 only
    if (blockIdx.x == 0 && threadIdx.x < head + tail) {
        const unsigned long long i = threadIdx.x < head
                                         ? threadIdx.x
                                         : (unsigned long long)head + n4 * 4ull + (threadIdx.x - head);
        int b;
        const uint32_t q = quantize_one<kScale>(in[i], p, b);
        if (kOut) out[i] = q;
        if (kStats) atomicAdd(&lane_hist[b * 32 + lane], 1u);
    }
    if (kStats) {
        __syncthreads();
        const int warp = threadIdx.x >> 5;
        for (int b = warp + 1; b < nbins; b += kThreads / 32) {  // bin 0 is never used
            const uint32_t c = __reduce_add_sync(0xFFFFFFFFu, lane_hist[b * 32 + lane]);
            if (lane == 0 && c != 0u) merge_bin(stats, p, b, c);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0 && n_total != 0ull)
            atomicAdd((unsigned long long*)&stats->n_total, n_total);
    }
}

// Any alignment: one element per thread per step.
template <bool kOut, bool kStats, bool kScale>
__global__ void __launch_bounds__(kThreads)
quantize_stats_scalar_kernel(const uint32_t* in, uint32_t* out, unsigned long long n,
                             QuantParams p, qfmt_stats_t* __restrict__ stats) {
    extern __shared__ uint32_t lane_hist[];
    const int nbins = p.top + kExtraBins;
    const int lane = threadIdx.x & 31;
    if (kStats) {
        for (int i = threadIdx.x; i < nbins * 32; i += kThreads) lane_hist[i] = 0u;
        __syncthreads();
    }
    const unsigned long long stride = (unsigned long long)gridDim.x * kThreads;
    for (unsigned long long i = (unsigned long long)blockIdx.x * kThreads + threadIdx.x; i < n; i += stride) {
        int b;
        const uint32_t q = quantize_one<kScale>(in[i], p, b);
        if (kOut) out[i] = q;
        if (kStats) atomicAdd(&lane_hist[b * 32 + lane], 1u);
    }
    if (kStats) {
        __syncthreads();
        const int warp = threadIdx.x >> 5;
        for (int b = warp + 1; b < nbins; b += kThreads / 32) {
            const uint32_t c = __reduce_add_sync(0xFFFFFFFFu, lane_hist[b * 32 + lane]);
            if (lane == 0 && c != 0u) merge_bin(stats, p, b, c);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0 && n != 0ull)
            atomicAdd((unsigned long long*)&stats->n_total, n);
    }
}

// Rounding with a batched transpose: in is [batch][rows][cols], out is [batch][cols][rows].
// 32 x 32 tiles go through shared memory so that both the reads (along cols) and the writes
// (along rows) are 128-byte segments; statistics as in the flat kernel.
constexpr int kTThreads = 256;
template <bool kStats, bool kScale>
__global__ void __launch_bounds__(kTThreads)
quantize_stats_transpose_kernel(const uint32_t* __restrict__ in, uint32_t* __restrict__ out, unsigned batch,
                                unsigned rows, unsigned cols, QuantParams p, qfmt_stats_t* __restrict__ stats,
                                unsigned long long n_total) {
    extern __shared__ uint32_t lane_hist[];  // [(top + kExtraBins)][32]
    __shared__ uint32_t tile[32][33];
    const int nbins = p.top + kExtraBins;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (kStats) {
        for (int i = threadIdx.x; i < nbins * 32; i += kTThreads) lane_hist[i] = 0u;
    }
    const unsigned tr = (rows + 31) / 32, tc = (cols + 31) / 32;
    const unsigned long long tiles = (unsigned long long)batch * tr * tc;
    for (unsigned long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        const unsigned b = (unsigned)(t / ((unsigned long long)tr * tc));
        const unsigned rem = (unsigned)(t % ((unsigned long long)tr * tc));
        const unsigned r0 = (rem / tc) * 32, c0 = (rem % tc) * 32;
        const unsigned long long base = (unsigned long long)b * rows * cols;
        __syncthreads();  // previous tile fully written out (and the histogram cleared)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const unsigned r = r0 + warp + 8 * i, c = c0 + lane;
            if (r < rows && c < cols) {
                int bin;
                const uint32_t q = quantize_one<kScale>(in[base + (unsigned long long)r * cols + c], p, bin);
                tile[warp + 8 * i][lane] = q;
                if (kStats) atomicAdd(&lane_hist[bin * 32 + lane], 1u);
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const unsigned c = c0 + warp + 8 * i, r = r0 + lane;
            if (r < rows && c < cols) out[base + (unsigned long long)c * rows + r] = tile[lane][warp + 8 * i];
        }
    }
    if (kStats) {
        __syncthreads();
        for (int b = warp + 1; b < nbins; b += kTThreads / 32) {
            const uint32_t c = __reduce_add_sync(0xFFFFFFFFu, lane_hist[b * 32 + lane]);
            if (lane == 0 && c != 0u) merge_bin(stats, p, b, c);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0 && n_total != 0ull)
            atomicAdd((unsigned long long*)&stats->n_total, n_total);
    }
}

QuantParams make_params(const qfmt_format_t& f) {
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
    return p;
}

template <bool kOut, bool kStats, bool kScale>
cudaError_t launch(const uint32_t* in, uint32_t* out, size_t n, const QuantParams& p, qfmt_stats_t* stats,
                   int sm_count, cudaStream_t stream) {
    const size_t smem = kStats ? (size_t)(p.top + kExtraBins) * 32 * sizeof(uint32_t) : 0;
    const uintptr_t ai = reinterpret_cast<uintptr_t>(in), ao = reinterpret_cast<uintptr_t>(out);
    const bool same_phase = !kOut || ((ai & 15u) == (ao & 15u));
    if (same_phase) {
        size_t head = ((16u - (ai & 15u)) & 15u) / 4u;
        if (head > n) head = n;
        const unsigned long long n4 = (n - head) / 4;
        const uint32_t tail = (uint32_t)((n - head) - n4 * 4);
        auto kern = quantize_stats_kernel<kOut, kStats, kScale>;
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        const unsigned long long per_block = (unsigned long long)kThreads * kUnroll;
        unsigned long long want = (n4 + per_block - 1) / per_block;
        // Measured on B200: 1024-1536 resident threads per SM stream faster than full occupancy,
        // and the 256-bin histogram (33 KB per block) must leave room for L1.
        const unsigned long long cap = (unsigned long long)sm_count * (p.top >= 255 ? 2 : 3);
        if (want > cap) want = cap;
        if (want == 0) want = 1;
        kern<<<(unsigned)want, kThreads, smem, stream>>>(in, out, (uint32_t)head, n4, tail, p, stats,
                                                         (unsigned long long)n);
    } else {
        auto kern = quantize_stats_scalar_kernel<kOut, kStats, kScale>;
        unsigned long long want = (n + kThreads - 1) / kThreads;
        const unsigned long long cap = (unsigned long long)sm_count * 4;
        if (want > cap) want = cap;
        if (want == 0) want = 1;
        kern<<<(unsigned)want, kThreads, smem, stream>>>(in, out, (unsigned long long)n, p, stats);
    }
    return cudaGetLastError();
}

}  // namespace

int quantize_stats_device(const float* d_in, float* d_out, size_t n, const qfmt_format_t* fmt,
                          qfmt_stats_t* d_stats, int accumulate, cudaStream_t stream) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    if (accumulate != 0 && accumulate != 1) return QFMT_ERR_BAD_ARG;
    if (n > ((size_t)1 << 40)) return QFMT_ERR_BAD_ARG;
    if (n != 0 && d_in == nullptr) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_in) & 3u) || (reinterpret_cast<uintptr_t>(d_out) & 3u) ||
        (reinterpret_cast<uintptr_t>(d_stats) & 7u))
        return QFMT_ERR_BAD_ARG;
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;
    if (d_stats != nullptr && accumulate == 0) QFMT_CUDA_TRY(cudaMemsetAsync(d_stats, 0, sizeof(qfmt_stats_t), stream));
    if (n == 0 || (d_out == nullptr && d_stats == nullptr)) return QFMT_OK;

    const QuantParams p = make_params(*fmt);
    const uint32_t* in = reinterpret_cast<const uint32_t*>(d_in);
    uint32_t* out = reinterpret_cast<uint32_t*>(d_out);
    const bool has_out = d_out != nullptr, has_stats = d_stats != nullptr, has_scale = fmt->loss_scale != 1.0f;
    cudaError_t err;
#define QFMT_DISPATCH(O, S, C) err = launch<O, S, C>(in, out, n, p, d_stats, dev.sm_count, stream)
    if (has_out && has_stats) { if (has_scale) QFMT_DISPATCH(true, true, true); else QFMT_DISPATCH(true, true, false); }
    else if (has_out) { if (has_scale) QFMT_DISPATCH(true, false, true); else QFMT_DISPATCH(true, false, false); }
    else { if (has_scale) QFMT_DISPATCH(false, true, true); else QFMT_DISPATCH(false, true, false); }
#undef QFMT_DISPATCH
    QFMT_CUDA_TRY(err);
    return QFMT_OK;
}


int quantize_stats_transpose_device(const float* d_in, float* d_out, int64_t batch, int64_t rows, int64_t cols,
                                    const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate,
                                    cudaStream_t stream) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    if (accumulate != 0 && accumulate != 1) return QFMT_ERR_BAD_ARG;
    if (batch < 0 || rows < 0 || cols < 0 || batch > 0x7FFFFFFF || rows > 0x7FFFFFFF || cols > 0x7FFFFFFF)
        return QFMT_ERR_BAD_ARG;
    const unsigned long long n = (unsigned long long)batch * (unsigned long long)rows * (unsigned long long)cols;
    if (n > (1ull << 40)) return QFMT_ERR_BAD_ARG;
    if (n != 0 && (d_in == nullptr || d_out == nullptr || d_in == d_out)) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_in) & 3u) || (reinterpret_cast<uintptr_t>(d_out) & 3u) ||
        (reinterpret_cast<uintptr_t>(d_stats) & 7u))
        return QFMT_ERR_BAD_ARG;
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;
    if (d_stats != nullptr && accumulate == 0) QFMT_CUDA_TRY(cudaMemsetAsync(d_stats, 0, sizeof(qfmt_stats_t), stream));
    if (n == 0) return QFMT_OK;
    const QuantParams p = make_params(*fmt);
    const uint32_t* in = reinterpret_cast<const uint32_t*>(d_in);
    uint32_t* out = reinterpret_cast<uint32_t*>(d_out);
    const bool has_stats = d_stats != nullptr, has_scale = fmt->loss_scale != 1.0f;
    const size_t smem = has_stats ? (size_t)(p.top + kExtraBins) * 32 * sizeof(uint32_t) : 0;
    const unsigned long long tiles = (unsigned long long)batch * ((rows + 31) / 32) * ((cols + 31) / 32);
    unsigned long long want = tiles < (unsigned long long)dev.sm_count * 8 ? tiles : (unsigned long long)dev.sm_count * 8;
#define QFMT_TLAUNCH(S, C)                                                                                       \
    quantize_stats_transpose_kernel<S, C><<<(unsigned)want, kTThreads, smem, stream>>>(                          \
        in, out, (unsigned)batch, (unsigned)rows, (unsigned)cols, p, d_stats, n)
    if (has_stats) { if (has_scale) QFMT_TLAUNCH(true, true); else QFMT_TLAUNCH(true, false); }
    else { if (has_scale) QFMT_TLAUNCH(false, true); else QFMT_TLAUNCH(false, false); }
#undef QFMT_TLAUNCH
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}

}  // namespace qfmt

extern "C" int qfmt_quantize_stats(const float* d_in, float* d_out, size_t n, const qfmt_format_t* fmt,
                                   qfmt_stats_t* d_stats, int accumulate, void* stream) {
    return qfmt::quantize_stats_device(d_in, d_out, n, fmt, d_stats, accumulate, (cudaStream_t)stream);
}

extern "C" int qfmt_quantize_stats_transpose(const float* d_in, float* d_out, int64_t batch, int64_t rows, int64_t cols,
                                             const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate,
                                             void* stream) {
    return qfmt::quantize_stats_transpose_device(d_in, d_out, batch, rows, cols, fmt, d_stats, accumulate,
                                                 (cudaStream_t)stream);
}

extern "C" size_t qfmt_quantize_stats_host_work_bytes(size_t n) {
    return ((n * sizeof(float) + 255u) & ~(size_t)255u) + sizeof(qfmt_stats_t);
}

extern "C" int qfmt_quantize_stats_host(const float* h_in, float* h_out, size_t n, const qfmt_format_t* fmt,
                                        qfmt_stats_t* h_stats, void* d_work, size_t work_bytes, void* stream_) {
    cudaStream_t stream = (cudaStream_t)stream_;
    if (n != 0 && h_in == nullptr) return QFMT_ERR_BAD_ARG;
    if (d_work == nullptr || (reinterpret_cast<uintptr_t>(d_work) & 15u)) return QFMT_ERR_BAD_ARG;
    if (work_bytes < qfmt_quantize_stats_host_work_bytes(n)) return QFMT_ERR_BAD_ARG;
    int rc = qfmt::validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    float* d_buf = reinterpret_cast<float*>(d_work);
    qfmt_stats_t* d_stats = reinterpret_cast<qfmt_stats_t*>(reinterpret_cast<char*>(d_work) +
                                                            ((n * sizeof(float) + 255u) & ~(size_t)255u));
    if (n) QFMT_CUDA_TRY(cudaMemcpyAsync(d_buf, h_in, n * sizeof(float), cudaMemcpyHostToDevice, stream));
    rc = qfmt::quantize_stats_device(d_buf, h_out ? d_buf : nullptr, n, fmt, h_stats ? d_stats : nullptr, 0, stream);
    if (rc != QFMT_OK) return rc;
    if (n && h_out) QFMT_CUDA_TRY(cudaMemcpyAsync(h_out, d_buf, n * sizeof(float), cudaMemcpyDeviceToHost, stream));
    if (h_stats) QFMT_CUDA_TRY(cudaMemcpyAsync(h_stats, d_stats, sizeof(qfmt_stats_t), cudaMemcpyDeviceToHost, stream));
    QFMT_CUDA_TRY(cudaStreamSynchronize(stream));
    return QFMT_OK;
}
