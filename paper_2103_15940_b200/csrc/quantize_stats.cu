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

#include <mutex>

#include "common.cuh"
#include "round.cuh"

namespace qfmt {
namespace {

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

__device__ __forceinline__ void store_stream(uint2* p, const uint2& v) {
    asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" :: "l"(p), "r"(v.x), "r"(v.y) : "memory");
}

constexpr int kThreads = 512;
constexpr int kUnroll = 4;  // 128-bit loads in flight per thread

// in/out point at the first element; `head` elements precede the 16-byte aligned body of n4
// vectors and `tail` elements follow it.
// kNative: 2 for bfloat16 (the vector body rounds by the hardware's conversion, see quantize_pair_native;
// 1 would be binary16, not instantiated), 0 for every other format.
template <bool kOut, bool kStats, bool kScale, int kNative>
__global__ void __launch_bounds__(kThreads)
quantize_stats_kernel(const uint32_t* in, uint32_t* out, uint32_t head,
                      unsigned long long n4, uint32_t tail, QuantParams p, qfmt_stats_t* __restrict__ stats,
                      unsigned long long n_total, const float* __restrict__ d_scale) {
    extern __shared__ uint32_t lane_hist[];  // [(top + kExtraBins)][32]
    grid_launch_dependents();  // a product launched after this pass may take the SMs as this grid leaves them
    if (kScale && d_scale != nullptr) p.scale = *d_scale;  // loss scale kept on the device (dynamic loss scaling)
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
                if (kNative) {
                    quantize_pair_native<kScale, kNative == 2>(v[u].x, v[u].y, p, q.x, q.y, b0, b1);
                    quantize_pair_native<kScale, kNative == 2>(v[u].z, v[u].w, p, q.z, q.w, b2, b3);
                } else {
                    q.x = quantize_one<kScale>(v[u].x, p, b0);
                    q.y = quantize_one<kScale>(v[u].y, p, b1);
                    q.z = quantize_one<kScale>(v[u].z, p, b2);
                    q.w = quantize_one<kScale>(v[u].w, p, b3);
                }
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
                             QuantParams p, qfmt_stats_t* __restrict__ stats, const float* __restrict__ d_scale) {
    extern __shared__ uint32_t lane_hist[];
    if (kScale && d_scale != nullptr) p.scale = *d_scale;
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

// 16-bit storage (Section II: activations and gradients are kept in 16 bits, halving storage and
// bandwidth): the rounding pass writing packed codes instead of fp32 containers, 4 bytes read and
// 2 written per element, and the pass that expands codes back to containers for the contraction.
// A thread takes eight consecutive elements: two 128-bit loads, one 128-bit store.
// kMode 1: results below the smallest normal are expected to be rare (formats with e >= 6): the denormal
// grid sits behind a branch (quantize_pack_one_rare_denormals).  kMode 2 / 3: binary16 / bfloat16 by the
// hardware's conversion in the vector body (quantize_pack_pair_native).  kMode 0: every other format.
template <bool kStats, bool kScale, int kMode>
__global__ void __launch_bounds__(kThreads)
quantize_stats_pack16_kernel(const uint32_t* __restrict__ in, uint16_t* __restrict__ codes, unsigned long long n,
                             int vec, QuantParams p, int sign_shift, qfmt_stats_t* __restrict__ stats) {
    extern __shared__ uint32_t lane_hist[];
    const int nbins = p.top + kExtraBins;
    const int lane = threadIdx.x & 31;
    if (kStats) {
        for (int i = threadIdx.x; i < nbins * 32; i += kThreads) lane_hist[i] = 0u;
        __syncthreads();
    }
    const unsigned long long n8 = vec ? n / 8 : 0ull;
    const unsigned long long stride = (unsigned long long)gridDim.x * (kThreads * 2);
    for (unsigned long long base = (unsigned long long)blockIdx.x * (kThreads * 2); base < n8; base += stride) {
        uint4 v[2][2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kThreads + threadIdx.x;
            if (idx < n8) {
                v[u][0] = load_stream(reinterpret_cast<const uint4*>(in) + 2 * idx);
                v[u][1] = load_stream(reinterpret_cast<const uint4*>(in) + 2 * idx + 1);
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const unsigned long long idx = base + (unsigned long long)u * kThreads + threadIdx.x;
            if (idx < n8) {
                const uint32_t w[8] = {v[u][0].x, v[u][0].y, v[u][0].z, v[u][0].w, v[u][1].x, v[u][1].y, v[u][1].z, v[u][1].w};
                if (kMode >= 2) {
                    uint32_t pk[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        int b0, b1;
                        pk[j] = quantize_pack_pair_native<kScale, kMode == 3>(w[2 * j], w[2 * j + 1], p, b0, b1);
                        if (kStats) {
                            atomicAdd(&lane_hist[b0 * 32 + lane], 1u);
                            atomicAdd(&lane_hist[b1 * 32 + lane], 1u);
                        }
                    }
                    store_stream(reinterpret_cast<uint4*>(codes) + idx, make_uint4(pk[0], pk[1], pk[2], pk[3]));
                } else {
                    uint32_t c[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        int b;
                        c[j] = kMode == 1 ? quantize_pack_one_rare_denormals<kScale>(w[j], p, sign_shift, b)
                                          : quantize_pack_one<kScale>(w[j], p, sign_shift, b);
                        if (kStats) atomicAdd(&lane_hist[b * 32 + lane], 1u);
                    }
                    store_stream(reinterpret_cast<uint4*>(codes) + idx,
                                 make_uint4(c[0] | (c[1] << 16), c[2] | (c[3] << 16), c[4] | (c[5] << 16), c[6] | (c[7] << 16)));
                }
            }
        }
    }
    // what the vector body leaves (everything when the pointers are not 16-byte aligned)
    const unsigned long long done = n8 * 8;
    for (unsigned long long i = done + (unsigned long long)blockIdx.x * kThreads + threadIdx.x; i < n;
         i += (unsigned long long)gridDim.x * kThreads) {
        int b;
        codes[i] = (uint16_t)(kMode == 1 ? quantize_pack_one_rare_denormals<kScale>(in[i], p, sign_shift, b)
                                         : quantize_pack_one<kScale>(in[i], p, sign_shift, b));
        if (kStats) atomicAdd(&lane_hist[b * 32 + lane], 1u);
    }
    if (kStats) {
        __syncthreads();
        const int warp = threadIdx.x >> 5;
        for (int b = warp + 1; b < nbins; b += kThreads / 32) {
            const uint32_t c = __reduce_add_sync(0xFFFFFFFFu, lane_hist[b * 32 + lane]);
            if (lane == 0 && c != 0u) merge_bin(stats, p, b, c);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0 && n != 0ull) atomicAdd((unsigned long long*)&stats->n_total, n);
    }
}

__global__ void __launch_bounds__(kThreads)
unpack16_kernel(const uint16_t* __restrict__ codes, uint32_t* __restrict__ out, unsigned long long n, int vec,
                QuantParams p, int sign_shift) {
    const unsigned long long n8 = vec ? n / 8 : 0ull;
    const unsigned long long stride = (unsigned long long)gridDim.x * kThreads;
    for (unsigned long long idx = (unsigned long long)blockIdx.x * kThreads + threadIdx.x; idx < n8; idx += stride) {
        const uint4 c = load_stream(reinterpret_cast<const uint4*>(codes) + idx);
        const uint32_t w[4] = {c.x, c.y, c.z, c.w};
        uint32_t q[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            q[2 * j] = unpack_one(w[j] & 0xFFFFu, p, sign_shift);
            q[2 * j + 1] = unpack_one(w[j] >> 16, p, sign_shift);
        }
        store_stream(reinterpret_cast<uint4*>(out) + 2 * idx, make_uint4(q[0], q[1], q[2], q[3]));
        store_stream(reinterpret_cast<uint4*>(out) + 2 * idx + 1, make_uint4(q[4], q[5], q[6], q[7]));
    }
    for (unsigned long long i = n8 * 8 + (unsigned long long)blockIdx.x * kThreads + threadIdx.x; i < n; i += stride)
        out[i] = unpack_one(codes[i], p, sign_shift);
}

// Layer output of Section IV-A's worked example, Y = R(R(acc) + R(B)): the matrix product is
// rounded, the (rounded) bias of its column is added, and the sum is rounded again, with the
// statistics of Y taken in the same pass.  The sum of two format values is formed with one IEEE
// fp32 add; for m <= 10 that add is either exact or so far from every grid and halfway point of
// the format that rounding its result equals rounding the exact sum (when the add is inexact the
// smaller term lies below 2^-12 of the larger one's last place).
// Vector kernel: rows of c4 = cols/4 128-bit vectors; each thread owns a column of vectors (its
// rounded bias entries stay in registers) and walks down the rows, four loads in flight.
// The same with 128-bit accesses on both sides, for rows and cols that are multiples of 4 and
// 16-byte aligned tensors: tiles of 64 rows x 32 columns; a thread loads four consecutive columns of
// a row (eight threads cover a 128-byte segment) and, after the exchange through shared memory,
// stores four consecutive rows of a column (sixteen threads cover the tile's 256 bytes of that
// output row).
constexpr int kTvRows = 64, kTvCols = 32;
template <bool kStats, bool kScale>
__global__ void __launch_bounds__(kTThreads)
quantize_stats_transpose_vec_kernel(const uint32_t* __restrict__ in, uint32_t* __restrict__ out, unsigned batch,
                                    unsigned rows, unsigned cols, QuantParams p, qfmt_stats_t* __restrict__ stats,
                                    unsigned long long n_total) {
    extern __shared__ uint32_t lane_hist[];  // [(top + kExtraBins)][32]
    __shared__ uint32_t tile[kTvRows][kTvCols + 1];
    const int nbins = p.top + kExtraBins;
    const int lane = threadIdx.x & 31;
    if (kStats) {
        for (int i = threadIdx.x; i < nbins * 32; i += kTThreads) lane_hist[i] = 0u;
    }
    const unsigned tr = (rows + kTvRows - 1) / kTvRows, tc = (cols + kTvCols - 1) / kTvCols;
    const unsigned long long tiles = (unsigned long long)batch * tr * tc;
    const unsigned lr = threadIdx.x / 8, lc4 = threadIdx.x % 8;    // load: row within a 32-row pass, column quad
    const unsigned sc = threadIdx.x / 16, sr4 = threadIdx.x % 16;  // store: column within a 16-column pass, row quad
    for (unsigned long long t = blockIdx.x; t < tiles; t += gridDim.x) {
        const unsigned b = (unsigned)(t / ((unsigned long long)tr * tc));
        const unsigned rem = (unsigned)(t % ((unsigned long long)tr * tc));
        const unsigned r0 = (rem / tc) * kTvRows, c0 = (rem % tc) * kTvCols;
        const unsigned long long base = (unsigned long long)b * rows * cols;
        uint4 v[2];
        bool ok[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const unsigned r = r0 + lr + 32 * i, c = c0 + 4 * lc4;
            ok[i] = r < rows && c < cols;
            if (ok[i]) v[i] = load_stream(reinterpret_cast<const uint4*>(in + base + (unsigned long long)r * cols + c));
        }
        __syncthreads();  // previous tile fully written out (and the histogram cleared)
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            if (ok[i]) {
                int b0, b1, b2, b3;
                uint32_t* dst = &tile[lr + 32 * i][4 * lc4];
                dst[0] = quantize_one<kScale>(v[i].x, p, b0);
                dst[1] = quantize_one<kScale>(v[i].y, p, b1);
                dst[2] = quantize_one<kScale>(v[i].z, p, b2);
                dst[3] = quantize_one<kScale>(v[i].w, p, b3);
                if (kStats) {
                    atomicAdd(&lane_hist[b0 * 32 + lane], 1u);
                    atomicAdd(&lane_hist[b1 * 32 + lane], 1u);
                    atomicAdd(&lane_hist[b2 * 32 + lane], 1u);
                    atomicAdd(&lane_hist[b3 * 32 + lane], 1u);
                }
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const unsigned c = c0 + sc + 16 * i, r = r0 + 4 * sr4;
            if (c < cols && r < rows) {
                uint4 q;
                q.x = tile[4 * sr4 + 0][sc + 16 * i];
                q.y = tile[4 * sr4 + 1][sc + 16 * i];
                q.z = tile[4 * sr4 + 2][sc + 16 * i];
                q.w = tile[4 * sr4 + 3][sc + 16 * i];
                store_stream(reinterpret_cast<uint4*>(out + base + (unsigned long long)c * rows + r), q);
            }
        }
    }
    if (kStats) {
        __syncthreads();
        const int warp = threadIdx.x >> 5;
        for (int b = warp + 1; b < nbins; b += kTThreads / 32) {
            const uint32_t c = __reduce_add_sync(0xFFFFFFFFu, lane_hist[b * 32 + lane]);
            if (lane == 0 && c != 0u) merge_bin(stats, p, b, c);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0 && n_total != 0ull)
            atomicAdd((unsigned long long*)&stats->n_total, n_total);
    }
}

template <bool kScale>
__device__ __forceinline__ uint32_t bias_round_one(uint32_t acc, uint32_t rb, const QuantParams& p, uint32_t inf_bits,
                                                   int& bin) {
    if (inf_bits != 0u) {
        const uint32_t ra = round_value<kScale>(acc, p, inf_bits);
        return round_sum(__float_as_uint(add_ieee(__uint_as_float(ra), __uint_as_float(rb))), p, bin);
    }
    // 1/8/m: values near fp32's largest would push the rounding constants out of range
    int unused;
    const uint32_t ra = quantize_one<kScale>(acc, p, unused);
    const uint32_t s = __float_as_uint(add_ieee(__uint_as_float(ra), __uint_as_float(rb)));
    const uint32_t q = quantize_one<false>(s, p, bin);
    // two finite terms whose fp32 sum is already infinite overflowed, they were not infinite
    if (bin == p.top + kBinInfIn && (ra & 0x7FFFFFFFu) < 0x7F800000u && (rb & 0x7FFFFFFFu) < 0x7F800000u)
        bin = p.top + kBinOverflow;
    return q;
}

// The common case of the layer formula in eleven float/integer operations per element: when the scaled
// product lies in a normal binade of the format below the top one, and so does the fp32 sum with the
// bias, neither rounding can overflow, underflow, lose a sign or meet a special value, and the result's
// bin is its own exponent field.  `ok` is cleared when either condition fails (the caller then takes
// the general path for the whole vector); lo2 = 2 * 2^E_min as a word shifted left by one (the sign
// drops out), span2 the width of the admitted exponent range in the same units.
template <bool kScale>
__device__ __forceinline__ uint32_t bias_round_fast(uint32_t acc, uint32_t rb, const QuantParams& p, uint32_t lo2,
                                                    uint32_t span2, bool& ok) {
    const uint32_t yb = kScale ? __float_as_uint(mul_ieee(__uint_as_float(acc), p.scale)) : acc;
    ok = ok && (((yb << 1) - lo2) < span2);
    const float c = __uint_as_float((yb & 0x7F800000u) + p.magic_add);
    const float ra = sub_ieee(add_ieee(__uint_as_float(yb), c), c);
    const uint32_t sb = __float_as_uint(add_ieee(ra, __uint_as_float(rb)));
    ok = ok && (((sb << 1) - lo2) < span2);
    const float c2 = __uint_as_float((sb & 0x7F800000u) + p.magic_add);
    return __float_as_uint(sub_ieee(add_ieee(__uint_as_float(sb), c2), c2));
}

// kPack: the output is written as packed 16-bit codes (out_v points at uint16_t, ld_out counts codes;
// four codes per 8-byte store) instead of fp32 containers.
template <bool kStats, bool kScale, bool kPack>
__global__ void __launch_bounds__(kThreads)
bias_quantize_stats_kernel(const uint32_t* acc, long long ld_acc, const uint32_t* __restrict__ bias, void* out_v,
                           long long ld_out, unsigned long long rows, uint32_t c4, uint32_t cw, uint32_t rpp,
                           QuantParams p, qfmt_stats_t* __restrict__ stats, int sign_shift) {
    uint32_t* const out = kPack ? nullptr : static_cast<uint32_t*>(out_v);
    uint16_t* const out16 = kPack ? static_cast<uint16_t*>(out_v) : nullptr;
    extern __shared__ uint32_t lane_hist[];  // [(top + kExtraBins)][32]
    const int nbins = p.top + kExtraBins;
    const int lane = threadIdx.x & 31;
    const uint32_t inf_bits = p.top < 255 ? (uint32_t)(p.top + p.code_off) << 23 : 0u;  // 2^(E_max+1); 0 = 1/8/m
    // fast path: exponent fields from E_min up to E_max - 1 (see bias_round_fast)
    const uint32_t lo2 = p.min_normal << 1, span2 = (inf_bits - (1u << 23) - p.min_normal) << 1;
    grid_dependency_wait();    // the sums come from the product launched before this pass
    grid_launch_dependents();
    if (kStats) {
        for (int i = threadIdx.x; i < nbins * 32; i += kThreads) lane_hist[i] = 0u;
        __syncthreads();
    }
    // A pass of the block covers rpp rows x cw vectors; a thread keeps its column, so the rounded
    // bias of that column stays in registers while it walks down the rows.
    const uint32_t r_local = threadIdx.x / cw, c_local = threadIdx.x % cw;
    if (r_local < rpp) {
        const unsigned long long row_step = (unsigned long long)gridDim.x * rpp;
        for (uint32_t cc = c_local; cc < c4; cc += cw) {
            const uint4 raw = reinterpret_cast<const uint4*>(bias)[cc];
            int unused;
            uint4 b;
            b.x = quantize_one<kScale>(raw.x, p, unused);
            b.y = quantize_one<kScale>(raw.y, p, unused);
            b.z = quantize_one<kScale>(raw.z, p, unused);
            b.w = quantize_one<kScale>(raw.w, p, unused);
            unsigned long long row = (unsigned long long)blockIdx.x * rpp + r_local;
            const uint4* pa = reinterpret_cast<const uint4*>(acc + row * ld_acc) + cc;
            uint4* po = kPack ? nullptr : reinterpret_cast<uint4*>(out + row * ld_out) + cc;
            uint2* po16 = kPack ? reinterpret_cast<uint2*>(out16 + row * ld_out) + cc : nullptr;
            const unsigned long long step_a = row_step * (unsigned long long)ld_acc / 4ull;  // in vectors
            const unsigned long long step_o = row_step * (unsigned long long)ld_out / 4ull;
            for (; row < rows; row += row_step * kUnroll) {
                uint4 v[kUnroll];
#pragma unroll
                for (int u = 0; u < kUnroll; ++u)
                    if (row + u * row_step < rows) v[u] = load_stream(pa + u * step_a);
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    if (row + u * row_step < rows) {
                        int b0, b1, b2, b3;
                        uint4 q;
                        bool ok = inf_bits != 0u;
                        if (ok) {
                            q.x = bias_round_fast<kScale>(v[u].x, b.x, p, lo2, span2, ok);
                            q.y = bias_round_fast<kScale>(v[u].y, b.y, p, lo2, span2, ok);
                            q.z = bias_round_fast<kScale>(v[u].z, b.z, p, lo2, span2, ok);
                            q.w = bias_round_fast<kScale>(v[u].w, b.w, p, lo2, span2, ok);
                            b0 = (int)((q.x >> 23) & 0xFFu) - p.code_off;
                            b1 = (int)((q.y >> 23) & 0xFFu) - p.code_off;
                            b2 = (int)((q.z >> 23) & 0xFFu) - p.code_off;
                            b3 = (int)((q.w >> 23) & 0xFFu) - p.code_off;
                        }
                        if (!ok) {
                            q.x = bias_round_one<kScale>(v[u].x, b.x, p, inf_bits, b0);
                            q.y = bias_round_one<kScale>(v[u].y, b.y, p, inf_bits, b1);
                            q.z = bias_round_one<kScale>(v[u].z, b.z, p, inf_bits, b2);
                            q.w = bias_round_one<kScale>(v[u].w, b.w, p, inf_bits, b3);
                        }
                        if (kPack) {
                            uint32_t c0, c1, c2, c3;
                            if (ok) {  // four normal results: re-biased fields shifted down, sign bit moved beside them
                                c0 = encode_normal(q.x, p, sign_shift); c1 = encode_normal(q.y, p, sign_shift);
                                c2 = encode_normal(q.z, p, sign_shift); c3 = encode_normal(q.w, p, sign_shift);
                            } else {
                                c0 = encode_container(q.x, b0, p, sign_shift); c1 = encode_container(q.y, b1, p, sign_shift);
                                c2 = encode_container(q.z, b2, p, sign_shift); c3 = encode_container(q.w, b3, p, sign_shift);
                            }
                            store_stream(po16 + u * step_o, make_uint2(c0 | (c1 << 16), c2 | (c3 << 16)));
                        } else {
                            store_stream(po + u * step_o, q);
                        }
                        if (kStats) {
                            atomicAdd(&lane_hist[b0 * 32 + lane], 1u);
                            atomicAdd(&lane_hist[b1 * 32 + lane], 1u);
                            atomicAdd(&lane_hist[b2 * 32 + lane], 1u);
                            atomicAdd(&lane_hist[b3 * 32 + lane], 1u);
                        }
                    }
                }
                pa += kUnroll * step_a;
                if (kPack) po16 += kUnroll * step_o; else po += kUnroll * step_o;
            }
        }
    }
    if (kStats) {
        __syncthreads();
        const int warp = threadIdx.x >> 5;
        for (int b = warp + 1; b < nbins; b += kThreads / 32) {
            const uint32_t c = __reduce_add_sync(0xFFFFFFFFu, lane_hist[b * 32 + lane]);
            if (lane == 0 && c != 0u) merge_bin(stats, p, b, c);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0)
            atomicAdd((unsigned long long*)&stats->n_total, rows * (unsigned long long)c4 * 4ull);
    }
}

// Any alignment and any column count: one element per thread per step, bias rounded per element.
template <bool kStats, bool kScale, bool kPack>
__global__ void __launch_bounds__(kThreads)
bias_quantize_stats_scalar_kernel(const uint32_t* acc, long long ld_acc, const uint32_t* __restrict__ bias,
                                  void* out_v, long long ld_out, unsigned long long rows, unsigned long long cols,
                                  QuantParams p, qfmt_stats_t* __restrict__ stats, int sign_shift) {
    extern __shared__ uint32_t lane_hist[];
    const int nbins = p.top + kExtraBins;
    const int lane = threadIdx.x & 31;
    if (kStats) {
        for (int i = threadIdx.x; i < nbins * 32; i += kThreads) lane_hist[i] = 0u;
        __syncthreads();
    }
    const unsigned long long n = rows * cols;
    const unsigned long long stride = (unsigned long long)gridDim.x * kThreads;
    const uint32_t inf_bits = p.top < 255 ? (uint32_t)(p.top + p.code_off) << 23 : 0u;
    for (unsigned long long i = (unsigned long long)blockIdx.x * kThreads + threadIdx.x; i < n; i += stride) {
        const unsigned long long r = i / cols, c = i % cols;
        int unused, b;
        const uint32_t rb = quantize_one<kScale>(bias[c], p, unused);
        const uint32_t q = bias_round_one<kScale>(acc[r * ld_acc + c], rb, p, inf_bits, b);
        if (kPack) static_cast<uint16_t*>(out_v)[r * ld_out + c] = (uint16_t)encode_container(q, p, sign_shift);
        else static_cast<uint32_t*>(out_v)[r * ld_out + c] = q;
        if (kStats) atomicAdd(&lane_hist[b * 32 + lane], 1u);
    }
    if (kStats) {
        __syncthreads();
        const int warp = threadIdx.x >> 5;
        for (int b = warp + 1; b < nbins; b += kThreads / 32) {
            const uint32_t c = __reduce_add_sync(0xFFFFFFFFu, lane_hist[b * 32 + lane]);
            if (lane == 0 && c != 0u) merge_bin(stats, p, b, c);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0 && n != 0ull) atomicAdd((unsigned long long*)&stats->n_total, n);
    }
}

template <bool kOut, bool kStats, bool kScale>
cudaError_t launch(const uint32_t* in, uint32_t* out, size_t n, const QuantParams& p, qfmt_stats_t* stats,
                   int sm_count, cudaStream_t stream, const float* d_scale, int native) {
    const size_t smem = kStats ? (size_t)(p.top + kExtraBins) * 32 * sizeof(uint32_t) : 0;
    const uintptr_t ai = reinterpret_cast<uintptr_t>(in), ao = reinterpret_cast<uintptr_t>(out);
    const bool same_phase = !kOut || ((ai & 15u) == (ao & 15u));
    if (same_phase) {
        size_t head = ((16u - (ai & 15u)) & 15u) / 4u;
        if (head > n) head = n;
        const unsigned long long n4 = (n - head) / 4;
        const uint32_t tail = (uint32_t)((n - head) - n4 * 4);
        auto kern = native == 2 ? quantize_stats_kernel<kOut, kStats, kScale, 2> : quantize_stats_kernel<kOut, kStats, kScale, 0>;
        if (smem > 48 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
        }
        const unsigned long long per_block = (unsigned long long)kThreads * kUnroll;
        unsigned long long want = (n4 + per_block - 1) / per_block;
        // Measured on B200: 1024-1536 resident threads per SM stream faster than full occupancy,
        // and the 256-bin histogram (33 KB per block) must leave room for L1.  With statistics three
        // blocks per SM hide the divergent zero/denormal path of denormal-heavy tensors (1/5/10 on
        // a tensor with half its values there: 99 us against 105 with two, 64 Mi elements); without them two blocks stream fastest (93 us).
        const unsigned long long cap = (unsigned long long)sm_count * ((kStats && p.top < 255) ? 3 : 2);
        if (want > cap) want = cap;
        if (want == 0) want = 1;
        kern<<<(unsigned)want, kThreads, smem, stream>>>(in, out, (uint32_t)head, n4, tail, p, stats,
                                                         (unsigned long long)n, d_scale);
    } else {
        auto kern = quantize_stats_scalar_kernel<kOut, kStats, kScale>;
        unsigned long long want = (n + kThreads - 1) / kThreads;
        const unsigned long long cap = (unsigned long long)sm_count * 4;
        if (want > cap) want = cap;
        if (want == 0) want = 1;
        kern<<<(unsigned)want, kThreads, smem, stream>>>(in, out, (unsigned long long)n, p, stats, d_scale);
    }
    return cudaGetLastError();
}

}  // namespace

int quantize_stats_device(const float* d_in, float* d_out, size_t n, const qfmt_format_t* fmt,
                          qfmt_stats_t* d_stats, int accumulate, cudaStream_t stream, const float* d_scale) {
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
    const bool has_out = d_out != nullptr, has_stats = d_stats != nullptr;
    const bool has_scale = fmt->loss_scale != 1.0f || d_scale != nullptr;
    cudaError_t err;
    // bfloat16 by the hardware's conversion (64 Mi elements: 95 us against 97.5).  binary16 could go the same
    // way (kNative = 1) but measured slower on tensors with many results below 2^-14, whose classification
    // then sits behind a divergent branch (102 us against 98), and no faster on the others.
    const int native = (fmt->e == 8 && fmt->m == 7) ? 2 : 0;
#define QFMT_DISPATCH(O, S, C) err = launch<O, S, C>(in, out, n, p, d_stats, dev.sm_count, stream, d_scale, native)
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
    const bool vec = (rows % 4 == 0) && (cols % 4 == 0) &&
                     !((reinterpret_cast<uintptr_t>(d_in) | reinterpret_cast<uintptr_t>(d_out)) & 15u);
    const unsigned long long tiles =
        vec ? (unsigned long long)batch * ((rows + kTvRows - 1) / kTvRows) * ((cols + kTvCols - 1) / kTvCols)
            : (unsigned long long)batch * ((rows + 31) / 32) * ((cols + 31) / 32);
    unsigned long long want = tiles < (unsigned long long)dev.sm_count * 8 ? tiles : (unsigned long long)dev.sm_count * 8;
#define QFMT_TLAUNCH(S, C)                                                                                       \
    do {                                                                                                         \
        if (vec)                                                                                                 \
            quantize_stats_transpose_vec_kernel<S, C><<<(unsigned)want, kTThreads, smem, stream>>>(              \
                in, out, (unsigned)batch, (unsigned)rows, (unsigned)cols, p, d_stats, n);                        \
        else                                                                                                     \
            quantize_stats_transpose_kernel<S, C><<<(unsigned)want, kTThreads, smem, stream>>>(                  \
                in, out, (unsigned)batch, (unsigned)rows, (unsigned)cols, p, d_stats, n);                        \
    } while (0)
    if (has_stats) { if (has_scale) QFMT_TLAUNCH(true, true); else QFMT_TLAUNCH(true, false); }
    else { if (has_scale) QFMT_TLAUNCH(false, true); else QFMT_TLAUNCH(false, false); }
#undef QFMT_TLAUNCH
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}


// pack: d_out points at 16-bit codes (ld_out counts codes) instead of fp32 containers.
int bias_quantize_stats_device(const float* d_acc, int64_t ld_acc, const float* d_bias, void* d_out, int64_t ld_out,
                               int64_t rows, int64_t cols, const qfmt_format_t* fmt, qfmt_stats_t* d_stats,
                               int accumulate, cudaStream_t stream, bool pack = false) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    if (fmt->m > 10) return QFMT_ERR_BAD_FORMAT;  // the one-add sum is only then a single rounding
    if (pack && fmt->e + fmt->m > 15) return QFMT_ERR_BAD_FORMAT;  // sign, exponent and mantissa must fit 16 bits
    if (accumulate != 0 && accumulate != 1) return QFMT_ERR_BAD_ARG;
    if (rows < 0 || cols < 0 || rows > ((int64_t)1 << 40) || cols > 0x7FFFFFFF) return QFMT_ERR_BAD_ARG;
    const unsigned long long n = (unsigned long long)rows * (unsigned long long)cols;
    if (n > (1ull << 40)) return QFMT_ERR_BAD_ARG;
    if (n != 0 && (d_acc == nullptr || d_bias == nullptr || d_out == nullptr)) return QFMT_ERR_BAD_ARG;
    if (n != 0 && (ld_acc < cols || ld_out < cols)) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_acc) & 3u) || (reinterpret_cast<uintptr_t>(d_out) & (pack ? 1u : 3u)) ||
        (reinterpret_cast<uintptr_t>(d_bias) & 3u) || (reinterpret_cast<uintptr_t>(d_stats) & 7u))
        return QFMT_ERR_BAD_ARG;
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;
    // cleared by a kernel that the pass behind it can overlap (see zero_words_kernel), not by a memset
    if (d_stats != nullptr && accumulate == 0)
        QFMT_CUDA_TRY(launch_overlapping(zero_words_kernel, 1u, 256u, 0, stream, reinterpret_cast<int*>(d_stats),
                                         (int)(sizeof(qfmt_stats_t) / sizeof(int))));
    if (n == 0) return QFMT_OK;

    const QuantParams p = make_params(*fmt);
    const uint32_t* acc = reinterpret_cast<const uint32_t*>(d_acc);
    const uint32_t* bias = reinterpret_cast<const uint32_t*>(d_bias);
    void* out = d_out;
    const int sign_shift = fmt->e + fmt->m;
    const bool has_stats = d_stats != nullptr, has_scale = fmt->loss_scale != 1.0f;
    const size_t hist_bytes = has_stats ? (size_t)(p.top + kExtraBins) * 32 * sizeof(uint32_t) : 0;
    // vector path: four elements per access, 16 bytes of fp32 and 8 bytes of codes
    const bool vec = (cols % 4 == 0) && (ld_acc % 4 == 0) && (ld_out % 4 == 0) &&
                     !((reinterpret_cast<uintptr_t>(d_acc) | reinterpret_cast<uintptr_t>(d_bias)) & 15u) &&
                     !(reinterpret_cast<uintptr_t>(d_out) & (pack ? 7u : 15u));
    cudaError_t err = cudaSuccess;
    if (vec) {
        const uint32_t c4 = (uint32_t)(cols / 4);
        const uint32_t cw = c4 < (uint32_t)kThreads ? c4 : (uint32_t)kThreads;  // vectors of a row per pass
        const uint32_t rpp = (uint32_t)kThreads / cw;                           // rows per pass
        const size_t smem = hist_bytes;
        unsigned long long want = ((unsigned long long)rows + (unsigned long long)rpp * kUnroll - 1) /
                                  ((unsigned long long)rpp * kUnroll);
        const unsigned long long cap = (unsigned long long)dev.sm_count * 2;  // 64 registers: two blocks per SM
        if (want > cap) want = cap;
#define QFMT_BLAUNCH(S, C, P)                                                                                     \
    err = launch_overlapping(bias_quantize_stats_kernel<S, C, P>, (unsigned)want, (unsigned)kThreads, smem, stream, \
        acc, (long long)ld_acc, bias, out, (long long)ld_out, (unsigned long long)rows, c4, cw, rpp, p, d_stats, sign_shift)
#define QFMT_BLAUNCH2(S, C) do { if (pack) QFMT_BLAUNCH(S, C, true); else QFMT_BLAUNCH(S, C, false); } while (0)
        if (has_stats) { if (has_scale) QFMT_BLAUNCH2(true, true); else QFMT_BLAUNCH2(true, false); }
        else { if (has_scale) QFMT_BLAUNCH2(false, true); else QFMT_BLAUNCH2(false, false); }
#undef QFMT_BLAUNCH2
#undef QFMT_BLAUNCH
    } else {
        unsigned long long want = (n + kThreads - 1) / kThreads;
        const unsigned long long cap = (unsigned long long)dev.sm_count * 4;
        if (want > cap) want = cap;
#define QFMT_BSLAUNCH(S, C, P)                                                                                     \
    bias_quantize_stats_scalar_kernel<S, C, P><<<(unsigned)want, kThreads, hist_bytes, stream>>>(                  \
        acc, (long long)ld_acc, bias, out, (long long)ld_out, (unsigned long long)rows, (unsigned long long)cols, p, d_stats, sign_shift)
#define QFMT_BSLAUNCH2(S, C) do { if (pack) QFMT_BSLAUNCH(S, C, true); else QFMT_BSLAUNCH(S, C, false); } while (0)
        if (has_stats) { if (has_scale) QFMT_BSLAUNCH2(true, true); else QFMT_BSLAUNCH2(true, false); }
        else { if (has_scale) QFMT_BSLAUNCH2(false, true); else QFMT_BSLAUNCH2(false, false); }
#undef QFMT_BSLAUNCH2
#undef QFMT_BSLAUNCH
    }
    QFMT_CUDA_TRY(err);
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}


int quantize_stats_pack16_device(const float* d_in, uint16_t* d_codes, size_t n, const qfmt_format_t* fmt,
                                 qfmt_stats_t* d_stats, int accumulate, cudaStream_t stream) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    if (fmt->e + fmt->m > 15) return QFMT_ERR_BAD_FORMAT;  // sign, exponent and mantissa must fit 16 bits
    if (accumulate != 0 && accumulate != 1) return QFMT_ERR_BAD_ARG;
    if (n > ((size_t)1 << 40)) return QFMT_ERR_BAD_ARG;
    if (n != 0 && (d_in == nullptr || d_codes == nullptr)) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_in) & 3u) || (reinterpret_cast<uintptr_t>(d_codes) & 1u) ||
        (reinterpret_cast<uintptr_t>(d_stats) & 7u))
        return QFMT_ERR_BAD_ARG;
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;
    if (d_stats != nullptr && accumulate == 0) QFMT_CUDA_TRY(cudaMemsetAsync(d_stats, 0, sizeof(qfmt_stats_t), stream));
    if (n == 0) return QFMT_OK;
    const QuantParams p = make_params(*fmt);
    const bool has_stats = d_stats != nullptr, has_scale = fmt->loss_scale != 1.0f;
    const size_t smem = has_stats ? (size_t)(p.top + kExtraBins) * 32 * sizeof(uint32_t) : 0;
    const int vec = !((reinterpret_cast<uintptr_t>(d_in) | reinterpret_cast<uintptr_t>(d_codes)) & 15u);
    const unsigned long long per_block = (unsigned long long)kThreads * 16;  // elements per block and sweep
    unsigned long long want = (n + per_block - 1) / per_block;
    const unsigned long long cap = (unsigned long long)dev.sm_count * 2;  // 56 registers x 512 threads: two per SM
    if (want > cap) want = cap;
    const uint32_t* in = reinterpret_cast<const uint32_t*>(d_in);
    const int sign_shift = fmt->e + fmt->m;
    // 1/5/m tensors of small gradients are mostly denormal (the paper's observation on binary16), so
    // only wider exponents take the kernel that branches on results below the smallest normal
    const int mode = (fmt->e == 5 && fmt->m == 10) ? 2 : (fmt->e == 8 && fmt->m == 7) ? 3 : (fmt->e >= 6 ? 1 : 0);
#define QFMT_PLAUNCH1(S, C, M) \
    quantize_stats_pack16_kernel<S, C, M><<<(unsigned)want, kThreads, smem, stream>>>(in, d_codes, n, vec, p, sign_shift, d_stats)
#define QFMT_PLAUNCH(S, C)                                                                                         \
    do {                                                                                                           \
        if (mode == 3) QFMT_PLAUNCH1(S, C, 3);                                                                     \
        else if (mode == 2) QFMT_PLAUNCH1(S, C, 2);                                                                \
        else if (mode == 1) QFMT_PLAUNCH1(S, C, 1);                                                                \
        else QFMT_PLAUNCH1(S, C, 0);                                                                               \
    } while (0)
    if (has_stats) { if (has_scale) QFMT_PLAUNCH(true, true); else QFMT_PLAUNCH(true, false); }
    else { if (has_scale) QFMT_PLAUNCH(false, true); else QFMT_PLAUNCH(false, false); }
#undef QFMT_PLAUNCH
#undef QFMT_PLAUNCH1
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}

int unpack16_device(const uint16_t* d_codes, float* d_out, size_t n, const qfmt_format_t* fmt, cudaStream_t stream) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    if (fmt->e + fmt->m > 15) return QFMT_ERR_BAD_FORMAT;
    if (n > ((size_t)1 << 40)) return QFMT_ERR_BAD_ARG;
    if (n != 0 && (d_codes == nullptr || d_out == nullptr)) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_codes) & 1u) || (reinterpret_cast<uintptr_t>(d_out) & 3u)) return QFMT_ERR_BAD_ARG;
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;
    if (n == 0) return QFMT_OK;
    const QuantParams p = make_params(*fmt);
    const int vec = !((reinterpret_cast<uintptr_t>(d_codes) | reinterpret_cast<uintptr_t>(d_out)) & 15u);
    unsigned long long want = (n / 8 + kThreads) / kThreads;
    const unsigned long long cap = (unsigned long long)dev.sm_count * 4;
    if (want > cap) want = cap;
    unpack16_kernel<<<(unsigned)want, kThreads, 0, stream>>>(d_codes, reinterpret_cast<uint32_t*>(d_out), n, vec, p,
                                                             fmt->e + fmt->m);
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}

}  // namespace qfmt

extern "C" int qfmt_quantize_stats(const float* d_in, float* d_out, size_t n, const qfmt_format_t* fmt,
                                   qfmt_stats_t* d_stats, int accumulate, void* stream) {
    return qfmt::quantize_stats_device(d_in, d_out, n, fmt, d_stats, accumulate, (cudaStream_t)stream, nullptr);
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

namespace qfmt {
namespace {

// Two helper streams per device for the host-buffer entry point: the copy to the device, the
// kernel and the copy back run on three streams so that the two directions of the link work at the
// same time.  Created on first use and kept until the process ends.
constexpr size_t kHostChunk = (size_t)2 << 20;  // elements per pipeline step (8 MiB)
struct HostPipe {
    cudaStream_t in = nullptr, out = nullptr;
};
int host_pipe(int ordinal, HostPipe* pipe) {
    static std::mutex mu;
    static HostPipe pipes[64];
    if (ordinal < 0 || ordinal >= 64) return QFMT_ERR_BAD_ARG;
    std::lock_guard<std::mutex> lock(mu);
    if (pipes[ordinal].in == nullptr) {
        HostPipe hp;
        QFMT_CUDA_TRY(cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking));
        QFMT_CUDA_TRY(cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking));
        pipes[ordinal] = hp;
    }
    *pipe = pipes[ordinal];
    return QFMT_OK;
}

}  // namespace
}  // namespace qfmt

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
    if (n <= qfmt::kHostChunk) {  // one piece: everything in order on the caller's stream
        if (n) QFMT_CUDA_TRY(cudaMemcpyAsync(d_buf, h_in, n * sizeof(float), cudaMemcpyHostToDevice, stream));
        rc = qfmt::quantize_stats_device(d_buf, h_out ? d_buf : nullptr, n, fmt, h_stats ? d_stats : nullptr, 0, stream,
                                         nullptr);
        if (rc != QFMT_OK) return rc;
        if (n && h_out) QFMT_CUDA_TRY(cudaMemcpyAsync(h_out, d_buf, n * sizeof(float), cudaMemcpyDeviceToHost, stream));
        if (h_stats) QFMT_CUDA_TRY(cudaMemcpyAsync(h_stats, d_stats, sizeof(qfmt_stats_t), cudaMemcpyDeviceToHost, stream));
        QFMT_CUDA_TRY(cudaStreamSynchronize(stream));
        return QFMT_OK;
    }
    // Pipeline over pieces of the tensor: piece i+1 travels to the device while piece i is rounded and
    // piece i-1 travels back.  Each piece has its own place in d_work, so nothing is overwritten.
    qfmt::DeviceInfo dev;
    rc = qfmt::current_device(&dev);
    if (rc != QFMT_OK) return rc;
    qfmt::HostPipe pipe;
    rc = qfmt::host_pipe(dev.ordinal, &pipe);
    if (rc != QFMT_OK) return rc;
    cudaEvent_t ev_in = nullptr, ev_k = nullptr;
    QFMT_CUDA_TRY(cudaEventCreateWithFlags(&ev_in, cudaEventDisableTiming));
    if (cudaEventCreateWithFlags(&ev_k, cudaEventDisableTiming) != cudaSuccess) {
        cudaEventDestroy(ev_in);
        return QFMT_ERR_CUDA;
    }
    cudaError_t err = cudaEventRecord(ev_k, stream);  // work already on the caller's stream comes first
    if (err == cudaSuccess) err = cudaStreamWaitEvent(pipe.in, ev_k, 0);
    if (err == cudaSuccess) err = cudaStreamWaitEvent(pipe.out, ev_k, 0);
    for (size_t off = 0, piece = 0; off < n && err == cudaSuccess && rc == QFMT_OK; off += qfmt::kHostChunk, ++piece) {
        const size_t len = n - off < qfmt::kHostChunk ? n - off : qfmt::kHostChunk;
        err = cudaMemcpyAsync(d_buf + off, h_in + off, len * sizeof(float), cudaMemcpyHostToDevice, pipe.in);
        if (err == cudaSuccess) err = cudaEventRecord(ev_in, pipe.in);
        if (err == cudaSuccess) err = cudaStreamWaitEvent(stream, ev_in, 0);
        if (err != cudaSuccess) break;
        rc = qfmt::quantize_stats_device(d_buf + off, h_out ? d_buf + off : nullptr, len, fmt, h_stats ? d_stats : nullptr,
                                         piece == 0 ? 0 : 1, stream, nullptr);
        if (rc != QFMT_OK) break;
        if (h_out) {
            err = cudaEventRecord(ev_k, stream);
            if (err == cudaSuccess) err = cudaStreamWaitEvent(pipe.out, ev_k, 0);
            if (err == cudaSuccess)
                err = cudaMemcpyAsync(h_out + off, d_buf + off, len * sizeof(float), cudaMemcpyDeviceToHost, pipe.out);
        }
    }
    if (err == cudaSuccess && rc == QFMT_OK && h_stats)
        err = cudaMemcpyAsync(h_stats, d_stats, sizeof(qfmt_stats_t), cudaMemcpyDeviceToHost, stream);
    // everything that was enqueued is waited for, also after an error, before the events go
    cudaError_t e1 = cudaStreamSynchronize(pipe.in), e2 = cudaStreamSynchronize(stream), e3 = cudaStreamSynchronize(pipe.out);
    cudaEventDestroy(ev_in);
    cudaEventDestroy(ev_k);
    if (rc != QFMT_OK) return rc;
    if (err == cudaSuccess) err = e1 != cudaSuccess ? e1 : (e2 != cudaSuccess ? e2 : e3);
    QFMT_CUDA_TRY(err);
    return QFMT_OK;
}

extern "C" int qfmt_bias_quantize_stats(const float* d_acc, int64_t ld_acc, const float* d_bias, float* d_out,
                                        int64_t ld_out, int64_t rows, int64_t cols, const qfmt_format_t* fmt,
                                        qfmt_stats_t* d_stats, int accumulate, void* stream) {
    return qfmt::bias_quantize_stats_device(d_acc, ld_acc, d_bias, d_out, ld_out, rows, cols, fmt, d_stats, accumulate,
                                            (cudaStream_t)stream);
}

extern "C" int qfmt_bias_quantize_stats_pack16(const float* d_acc, int64_t ld_acc, const float* d_bias, uint16_t* d_codes,
                                               int64_t ld_codes, int64_t rows, int64_t cols, const qfmt_format_t* fmt,
                                               qfmt_stats_t* d_stats, int accumulate, void* stream) {
    return qfmt::bias_quantize_stats_device(d_acc, ld_acc, d_bias, d_codes, ld_codes, rows, cols, fmt, d_stats, accumulate,
                                            (cudaStream_t)stream, true);
}

extern "C" int qfmt_quantize_stats_pack16(const float* d_in, uint16_t* d_codes, size_t n, const qfmt_format_t* fmt,
                                          qfmt_stats_t* d_stats, int accumulate, void* stream) {
    return qfmt::quantize_stats_pack16_device(d_in, d_codes, n, fmt, d_stats, accumulate, (cudaStream_t)stream);
}

extern "C" int qfmt_unpack16(const uint16_t* d_codes, float* d_out, size_t n, const qfmt_format_t* fmt, void* stream) {
    return qfmt::unpack16_device(d_codes, d_out, n, fmt, (cudaStream_t)stream);
}
