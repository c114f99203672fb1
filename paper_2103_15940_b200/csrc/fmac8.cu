// FMAC-8 matrix product (Algorithm 1): every output is a dot product accumulated with FMAC
// instructions, a16 = round(a16 + x16 * y16) with ONE rounding to the 16-bit format
// (Section III-B), in groups of eight; each group's sum is added to a single-precision master
// accumulator with an fp32 add and the small accumulator restarts from zero; the master
// accumulator is rounded to the format at the end.  Statistics of the output tensor are taken
// in the same kernel.
//
// No tensor core implements "round the accumulator to 11 bits after every product", so this is
// plain-ALU work (a few dozen integer/float instructions per multiply-add, or one HFMA2 per two
// multiply-adds for binary16, which the ALUs implement natively); operand traffic is negligible
// beside it.  Two kernels:
//   * fmac8_kernel, any format with m <= 10.  The exact value a + x*y is rounded ONCE by forming
//     it to 24 bits with round-to-odd (the two directed fp32 fused multiply-adds; when they differ
//     the one with an odd last bit is taken) and then rounding to m+1 bits to nearest-even: a
//     sticky last bit 13 or more places below the target's last place cannot create or hide a tie.
//   * fmac8_f16_kernel, 1/5/10 and 1/8/7: fma.rn.f16x2 and fma.rn.bf16x2 are this very operation
//     for IEEE binary16 and for bfloat16 with denormals; flushing formats clear results below the
//     smallest normal afterwards.
// They keep a 64 x 64 (resp. 64 x 128) tile of outputs per block in registers and stream
// 32-deep slices of the operands through shared memory.
//
// Convolution layers (Section IV-A: FMAC-8 also names a convolution whose sums are accumulated this
// way).  The three products of a unit-stride, zero-padded convolution on channels-last tensors run on
// the same kernels (their kConv instantiations) as matrix products whose activation-like operand is
// gathered at the filter taps' offsets while a slice is staged; a position in the padding is a zero
// factor that keeps its place in its run of eight.  Order of the reduction index (the paper leaves it
// open; this is the order of the unfolded channels-last operand matrix):
//   forward          taps (r, then s), within a tap the input channels
//   data gradient    taps (r, then s), within a tap the output channels
//   filter gradient  images, within an image the output rows, within a row the output pixels
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"
#include "round.cuh"

namespace qfmt {
namespace {

constexpr int kFmThreads = 256;
constexpr int kFmBK = 32;    // K elements per shared-memory slice: four groups of eight
constexpr int kGroup = 8;    // FMACs per group (Algorithm 1)

// How the gathered operand of a convolution product is addressed.  A pixel index runs over
// [image][PH][PW]; a tap-and-channel index is tap * C + channel with tap = r * S + s.  The element for
// pixel (b, y, x) and (r, s, c) is src[((b * H + y + sign * r + off_h) * W + x + sign * s + off_w) * C + c],
// zero when that row or column lies outside the tensor.
struct ConvGather {
    int mode;             // 0 plain matrices, 1 forward, 2 data gradient, 3 filter gradient
    int H, W, C;          // the gathered tensor [n][H][W][C]
    int PH, PW, pixels;   // the pixel space and its size n * PH * PW
    int S, taps;          // filter taps per row, taps in all
    int sign, off_h, off_w;
    int filt_n, filt_k;   // data gradient: filters [filt_k = c_out][taps][filt_n = c_in]
    int vec4;             // both channel counts are multiples of four and the tensors 16-byte aligned:
                          // four consecutive channels are one 128-bit load
};

struct FmacParams {
    const float* A;
    const float* B;
    float* C;
    long long lda, ldb, ldc;
    int M, N, K;
    int transA, transB;
    int vec_store;  // C rows 16-byte aligned
    int vec_a, vec_b;  // operand base and leading dimension allow 128-bit loads
    ConvGather cv;
};

// Table entries of the gather: a pixel as {offset of its image, y, x, inside the pixel space}, a
// tap-and-channel index as {row offset, column offset, channel, inside the index range}.
__device__ __forceinline__ int4 pixel_entry(const ConvGather& cv, int pix) {
    const int x = pix % cv.PW, q = pix / cv.PW;
    return make_int4((q / cv.PH) * cv.H * cv.W * cv.C, q % cv.PH, x, pix < cv.pixels ? 1 : 0);
}
__device__ __forceinline__ int4 tap_entry(const ConvGather& cv, int tc) {
    const int c = tc % cv.C, tap = tc / cv.C;
    return make_int4(cv.sign * (tap / cv.S) + cv.off_h, cv.sign * (tap % cv.S) + cv.off_w, c, tap < cv.taps ? 1 : 0);
}
__device__ __forceinline__ float gather_element(const ConvGather& cv, const float* src, const int4& px, const int4& tc) {
    const int ih = px.y + tc.x, iw = px.z + tc.y;
    if (!(px.w & tc.w) || (unsigned)ih >= (unsigned)cv.H || (unsigned)iw >= (unsigned)cv.W) return 0.0f;
    return src[px.x + (ih * cv.W + iw) * cv.C + tc.z];
}
// Data gradient: offset of filter row k = tap * c_out + o, i.e. of W[o][tap][0], or -1 past the end.
__device__ __forceinline__ int filter_row_entry(const ConvGather& cv, int k) {
    const int o = k % cv.filt_k, tap = k / cv.filt_k;
    return tap < cv.taps ? (o * cv.taps + tap) * cv.filt_n : -1;
}
// Tables of a convolution product in shared memory: 64 pixels or 32, 128 tap-and-channel indices or 32.
struct ConvTables {
    int4 pix[64];
    int4 tap[128];
    int filt[kFmBK];
};
// Per tile (slice = false) and per slice (slice = true): the entries that depend on the tile's rows /
// columns, and those that depend on the slice's k range.  kCols is the tile's width.
template <int kRows, int kCols>
__device__ __forceinline__ void conv_tables(ConvTables& t, const ConvGather& cv, bool slice, int m0, int n0, int k0) {
    const int i = threadIdx.x;
    if (!slice) {
        if (cv.mode != 3) { if (i < kRows) t.pix[i] = pixel_entry(cv, m0 + i); }
        else if (i < kCols) t.tap[i] = tap_entry(cv, n0 + i);
    } else if (i < kFmBK) {
        if (cv.mode != 3) t.tap[i] = tap_entry(cv, k0 + i);
        else t.pix[i] = pixel_entry(cv, k0 + i);
        if (cv.mode == 2) t.filt[i] = filter_row_entry(cv, k0 + i);
    }
}
// A convolution's slice of op(A) (kIsA) or op(B) as [k][row or column], converted by `convert`.
template <int kRows, int kLd, bool kIsA, typename T, typename F>
__device__ __forceinline__ void load_slice_conv(T (*dst)[kLd], const FmacParams& g, const ConvTables& t, int r0, int k0,
                                                F convert) {
    const ConvGather& cv = g.cv;
    const bool gathered = kIsA ? cv.mode != 3 : cv.mode == 3;
    for (int idx = threadIdx.x; idx < kRows * kFmBK; idx += kFmThreads) {
        float v;
        int r, k;
        if (gathered && kIsA) {            // consecutive k are consecutive channels of a pixel
            k = idx % kFmBK; r = idx / kFmBK;
            v = gather_element(cv, g.A, t.pix[r], t.tap[k]);
        } else if (gathered) {             // filter gradient: consecutive columns are consecutive channels
            r = idx % kRows; k = idx / kRows;
            v = gather_element(cv, g.B, t.pix[k], t.tap[r]);
        } else if (kIsA) {                 // filter gradient: dY as [pixel][c_out], op(A)[i][k] = dY[k][i]
            r = idx % kRows; k = idx / kRows;
            v = (r0 + r < g.M && k0 + k < g.K) ? g.A[(long long)(k0 + k) * g.lda + (r0 + r)] : 0.0f;
        } else if (cv.mode == 1) {         // forward: filters [c_out][taps * c_in], k contiguous
            k = idx % kFmBK; r = idx / kFmBK;
            v = (r0 + r < g.N && k0 + k < g.K) ? g.B[(long long)(r0 + r) * g.ldb + (k0 + k)] : 0.0f;
        } else {                           // data gradient: filters [c_out][taps][c_in], row k = (tap, c_out)
            r = idx % kRows; k = idx / kRows;
            v = (t.filt[k] >= 0 && r0 + r < g.N) ? g.B[t.filt[k] + r0 + r] : 0.0f;
        }
        dst[k][r] = convert(v);
    }
}

// a + x*y rounded to 24 bits with round-to-odd.  The two directed fused multiply-adds (exact
// product, one rounding) are equal when the value is exact and adjacent fp32 numbers otherwise,
// exactly one of which has an odd last bit.  (An exact cancellation gives -0 and +0; the
// even-looking -0 loses, so +0 comes out as in round-to-nearest.)  Nothing is required of the
// product's range: beyond fp32's largest the pair is (largest, inf) and the odd "largest" rounds
// to the format's infinity afterwards; below its smallest denormal the pair is (0, 2^-149) and the
// odd 2^-149 is a sticky bit far below every format's quantum.
__device__ __forceinline__ uint32_t fma_to_odd(float a, float x, float y) {
    float lo, hi;
    asm("fma.rm.f32 %0, %1, %2, %3;" : "=f"(lo) : "f"(x), "f"(y), "f"(a));
    asm("fma.rp.f32 %0, %1, %2, %3;" : "=f"(hi) : "f"(x), "f"(y), "f"(a));
    const uint32_t l = __float_as_uint(lo), h = __float_as_uint(hi);
    return (l & 1u) ? l : h;
}

struct SmallRound {
    uint32_t min_normal;  // fp32 bits of 2^E_min
    uint32_t inf_bits;    // fp32 bits of 2^(E_max+1) (of +inf for e = 8)
    uint32_t magic_add;   // ((23 - m) << 23) | 0x400000
    uint32_t big_exp;     // e = 8: exponent fields above this one take the integer rounding
    uint32_t drop, round_add, keep_mask;
};

// Rounds a 24-bit intermediate to the format (the small accumulator's rounding; no statistics).
// With C = 1.5 * 2^(max(floor(log2|s|), E_min) + 23 - m), the fp32 sum s + C stays in C's binade,
// whose last place is the format's quantum for s, so (s + C) - C is s rounded to nearest-even on
// the format's grid, normal or denormal, either sign (a zero result may come out as +0 where -0 is
// meant; nothing downstream can tell: it is only ever added to other numbers).  kWide = 1 (e = 7):
// a + x*y can approach 2^128, so the exponent is capped at E_max+1 to keep C finite; whatever
// reaches 2^(E_max+1) is made infinite afterwards.  kWide = 2 (e = 8): values up to fp32's largest
// are values of the format, and near the top C would leave fp32's range; those few take the
// integer rounding of the fp32 word instead.
template <bool kFlush, int kWide>
__device__ __forceinline__ float round_small(uint32_t s, const SmallRound& r) {
    uint32_t ec = s & 0x7F800000u;
    float q;
    if (kWide == 2 && ec > r.big_exp) {
        const uint32_t a = s & 0x7FFFFFFFu;
        const uint32_t qa = a > 0x7F800000u ? 0x7FC00000u : ((a + r.round_add + ((a >> r.drop) & 1u)) & r.keep_mask);
        q = __uint_as_float((s & 0x80000000u) | qa);
    } else {
        ec = ec < r.min_normal ? r.min_normal : ec;
        if (kWide == 1) ec = ec > r.inf_bits ? r.inf_bits : ec;
        const float c = __uint_as_float(ec + r.magic_add);
        q = sub_ieee(add_ieee(__uint_as_float(s), c), c);
    }
    if (!(fabsf(q) < __uint_as_float(r.inf_bits)))
        q = (q != q) ? __uint_as_float(0x7FC00000u) : copysignf(__uint_as_float(0x7F800000u), q);
    if (kFlush && fabsf(q) < __uint_as_float(r.min_normal)) q = 0.0f;
    return q;
}

template <bool kFlush, int kWide>
__device__ __forceinline__ float fmac(float acc, float x, float y, const SmallRound& r) {
    return round_small<kFlush, kWide>(fma_to_odd(acc, x, y), r);
}

// One 32-deep slice of op(A) (rows m0.., kBM of them) into shared memory as [k][m]; elements
// outside the matrix are zero (a zero product leaves a format-valued accumulator unchanged).
template <int kRows, int kLd, typename T, typename F>
__device__ __forceinline__ void load_slice(T (*dst)[kLd], const float* src, long long ld, int trans_k_major,
                                           int r0, int rmax, int k0, int kmax, F convert) {
    // trans_k_major != 0: k is the contiguous index of the stored matrix
    for (int idx = threadIdx.x; idx < kRows * kFmBK; idx += kFmThreads) {
        int r, k;
        if (trans_k_major) { k = idx % kFmBK; r = idx / kFmBK; }
        else { r = idx % kRows; k = idx / kRows; }
        float v = 0.0f;
        if (r0 + r < rmax && k0 + k < kmax)
            v = trans_k_major ? src[(long long)(r0 + r) * ld + (k0 + k)] : src[(long long)(k0 + k) * ld + (r0 + r)];
        dst[k][r] = convert(v);
    }
}

// Rounds the master accumulators of one thread's rows x cols patch, stores them and counts.
template <bool kStats, int kTM, int kTN>
__device__ __forceinline__ void store_patch(const FmacParams& g, const QuantParams& p, const float (&master)[kTM][kTN],
                                            int row0, int col0, uint32_t* lane_hist, int lane) {
#pragma unroll
    for (int i = 0; i < kTM; ++i) {
        const int row = row0 + i;
        if (row >= g.M) break;
        uint32_t q[kTN];
#pragma unroll
        for (int j = 0; j < kTN; ++j) {
            int bin;
            q[j] = quantize_one<false>(__float_as_uint(master[i][j]), p, bin);
            if (kStats && col0 + j < g.N) atomicAdd(&lane_hist[bin * 32 + lane], 1u);
        }
        float* dst = g.C + (long long)row * g.ldc + col0;
#pragma unroll
        for (int j = 0; j < kTN; j += 4) {
            if (g.vec_store && col0 + j + 3 < g.N) {
                *reinterpret_cast<uint4*>(dst + j) = make_uint4(q[j], q[j + 1], q[j + 2], q[j + 3]);
            } else {
#pragma unroll
                for (int jj = j; jj < j + 4; ++jj)
                    if (col0 + jj < g.N) dst[jj] = __uint_as_float(q[jj]);
            }
        }
    }
}

template <bool kStats>
__device__ __forceinline__ void merge_block_hist(qfmt_stats_t* stats, const QuantParams& p, uint32_t* lane_hist,
                                                 int nbins, unsigned long long n_total) {
    if (!kStats) return;
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int b = warp + 1; b < nbins; b += kFmThreads / 32) {
        const uint32_t c = __reduce_add_sync(0xFFFFFFFFu, lane_hist[b * 32 + lane]);
        if (lane == 0 && c != 0u) merge_bin(stats, p, b, c);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0 && n_total != 0ull)
        atomicAdd((unsigned long long*)&stats->n_total, n_total);
}

// The same with 128-bit loads (ConvGather::vec4): a group is four consecutive channels, which are four
// consecutive k of a pixel (forward / data gradient: gathered operand and forward filters), or four
// consecutive rows or columns of a k (the other operands).  Channel counts that are multiples of four
// keep a group inside one tap, inside the matrix, and 16-byte aligned.
template <int kRows, int kLd, bool kIsA, typename T, typename F>
__device__ __forceinline__ void load_slice_conv4(T (*dst)[kLd], const FmacParams& g, const ConvTables& t, int r0, int k0,
                                                 F convert) {
    const ConvGather& cv = g.cv;
    const bool gathered = kIsA ? cv.mode != 3 : cv.mode == 3;
    const bool along_k = kIsA ? cv.mode != 3 : cv.mode == 1;
    const float* src = kIsA ? g.A : g.B;
    for (int idx = threadIdx.x; idx < kRows * kFmBK / 4; idx += kFmThreads) {
        int r, k;
        if (along_k) { k = 4 * (idx % (kFmBK / 4)); r = idx / (kFmBK / 4); }
        else { r = 4 * (idx % (kRows / 4)); k = idx / (kRows / 4); }
        const float* ptr = nullptr;
        if (gathered) {
            const int4 px = kIsA ? t.pix[r] : t.pix[k], tc = kIsA ? t.tap[k] : t.tap[r];
            const int ih = px.y + tc.x, iw = px.z + tc.y;
            if ((px.w & tc.w) && (unsigned)ih < (unsigned)cv.H && (unsigned)iw < (unsigned)cv.W)
                ptr = src + px.x + (ih * cv.W + iw) * cv.C + tc.z;
        } else if (kIsA) {            // filter gradient: op(A)[i][k] = dY[k][i]
            if (r0 + r < g.M && k0 + k < g.K) ptr = src + (long long)(k0 + k) * g.lda + (r0 + r);
        } else if (cv.mode == 1) {    // forward: filters [c_out][taps * c_in]
            if (r0 + r < g.N && k0 + k < g.K) ptr = src + (long long)(r0 + r) * g.ldb + (k0 + k);
        } else {                      // data gradient: filters [c_out][taps][c_in]
            if (t.filt[k] >= 0 && r0 + r < g.N) ptr = src + t.filt[k] + r0 + r;
        }
        const float4 v = ptr != nullptr ? *reinterpret_cast<const float4*>(ptr) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        if (along_k) {
            dst[k][r] = convert(v.x); dst[k + 1][r] = convert(v.y); dst[k + 2][r] = convert(v.z); dst[k + 3][r] = convert(v.w);
        } else {
            dst[k][r] = convert(v.x); dst[k][r + 1] = convert(v.y); dst[k][r + 2] = convert(v.z); dst[k][r + 3] = convert(v.w);
        }
    }
}

// ---- any format with m <= 10 ----------------------------------------------------------------
// 4 x 4 outputs per thread: the FMAC chain of one output is a dozen dependent instructions, so
// many resident warps (four blocks per SM) hide more latency than a larger patch per thread would.
constexpr int kFmBM = 64, kFmBN = 64, kFmTM = 4, kFmTN = 4;
constexpr int kFmBlocksPerSm = 4;

template <bool kStats, bool kFlush, int kWide, bool kConv>
__global__ void __launch_bounds__(kFmThreads, kFmBlocksPerSm)
fmac8_kernel(FmacParams g, QuantParams p, qfmt_stats_t* __restrict__ stats) {
    __shared__ __align__(16) float As[kFmBK][kFmBM + 4];
    __shared__ __align__(16) float Bs[kFmBK][kFmBN + 4];
    __shared__ ConvTables tabs[1];  // used by the convolution instantiations only
    extern __shared__ uint32_t lane_hist[];  // [(top + kExtraBins)][32]
    const int nbins = p.top + kExtraBins;
    const int lane = threadIdx.x & 31;
    if (kStats) {
        for (int i = threadIdx.x; i < nbins * 32; i += kFmThreads) lane_hist[i] = 0u;
        __syncthreads();
    }
    SmallRound sr;
    sr.min_normal = p.min_normal;
    sr.inf_bits = (uint32_t)(p.top + p.code_off) << 23;
    sr.magic_add = p.magic_add;
    sr.big_exp = (254u - p.drop) << 23;
    sr.drop = p.drop;
    sr.round_add = p.round_add;
    sr.keep_mask = p.keep_mask;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const int tiles_n = (g.N + kFmBN - 1) / kFmBN, tiles_m = (g.M + kFmBM - 1) / kFmBM;
    auto same = [](float v) { return v; };
    for (long long tile = blockIdx.x; tile < (long long)tiles_m * tiles_n; tile += gridDim.x) {
        const int m0 = (int)(tile / tiles_n) * kFmBM, n0 = (int)(tile % tiles_n) * kFmBN;
        float master[kFmTM][kFmTN], small[kFmTM][kFmTN];
#pragma unroll
        for (int i = 0; i < kFmTM; ++i)
#pragma unroll
            for (int j = 0; j < kFmTN; ++j) master[i][j] = 0.0f, small[i][j] = 0.0f;
        if (kConv) conv_tables<kFmBM, kFmBN>(tabs[0], g.cv, false, m0, n0, 0);  // read after the next barrier
        for (int k0 = 0; k0 < g.K; k0 += kFmBK) {
            __syncthreads();  // the previous slice is no longer read
            if (kConv) {
                conv_tables<kFmBM, kFmBN>(tabs[0], g.cv, true, m0, n0, k0);
                __syncthreads();
                if (g.cv.vec4) {
                    load_slice_conv4<kFmBM, kFmBM + 4, true>(As, g, tabs[0], m0, k0, same);
                    load_slice_conv4<kFmBN, kFmBN + 4, false>(Bs, g, tabs[0], n0, k0, same);
                } else {
                    load_slice_conv<kFmBM, kFmBM + 4, true>(As, g, tabs[0], m0, k0, same);
                    load_slice_conv<kFmBN, kFmBN + 4, false>(Bs, g, tabs[0], n0, k0, same);
                }
            } else {
                load_slice<kFmBM, kFmBM + 4>(As, g.A, g.lda, !g.transA, m0, g.M, k0, g.K, same);
                load_slice<kFmBN, kFmBN + 4>(Bs, g.B, g.ldb, g.transB, n0, g.N, k0, g.K, same);
            }
            __syncthreads();
            const int kmax = g.K - k0 < kFmBK ? g.K - k0 : kFmBK;
#pragma unroll 1
            for (int kg = 0; kg < kmax; kg += kGroup) {
#pragma unroll
                for (int kk = 0; kk < kGroup; ++kk) {
                    const float4 a0 = *reinterpret_cast<const float4*>(&As[kg + kk][ty * kFmTM]);
                    const float4 b0 = *reinterpret_cast<const float4*>(&Bs[kg + kk][tx * kFmTN]);
                    const float a[kFmTM] = {a0.x, a0.y, a0.z, a0.w};
                    const float b[kFmTN] = {b0.x, b0.y, b0.z, b0.w};
#pragma unroll
                    for (int i = 0; i < kFmTM; ++i)
#pragma unroll
                        for (int j = 0; j < kFmTN; ++j) small[i][j] = fmac<kFlush, kWide>(small[i][j], a[i], b[j], sr);
                }
                // the group's sum moves to the master accumulator (fp32 addition)
#pragma unroll
                for (int i = 0; i < kFmTM; ++i)
#pragma unroll
                    for (int j = 0; j < kFmTN; ++j) {
                        master[i][j] = add_ieee(master[i][j], small[i][j]);
                        small[i][j] = 0.0f;
                    }
            }
        }
        store_patch<kStats, kFmTM, kFmTN>(g, p, master, m0 + ty * kFmTM, n0 + tx * kFmTN, lane_hist, lane);
    }
    merge_block_hist<kStats>(stats, p, lane_hist, nbins, (unsigned long long)g.M * (unsigned long long)g.N);
}

// ---- 1/5/10 and 1/8/7: the hardware's own 16-bit fused multiply-adds --------------------------
constexpr int kHfBM = 64, kHfBN = 128, kHfTM = 4, kHfTN = 8;
// Resident blocks per SM: two for matrix products (the next operand slice waits in registers while this one
// is used: 120 registers a thread), three for convolutions (their gathered slices are not fetched ahead, so
// a third block hides more of the gather: 14.3 -> 15.5 TFMAC/s on a 3 x 3 layer, where matrix products lose:
// 19.7 -> 18.5).
constexpr int kHfBlocksPerSm = 2, kHfConvBlocksPerSm = 3;

// two FMACs: {a.lo * b.lo + c.lo, a.hi * b.hi + c.hi}, each rounded once to the 16-bit type
template <bool kBf16>
__device__ __forceinline__ uint32_t fma2_16(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    if (kBf16) asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    else asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));  // no .ftz: denormals honoured
    return r;
}

// clears the 16-bit halves whose magnitude is below the smallest normal (0x0400 = 2^-14 for
// binary16, 0x0080 = 2^-126 for bfloat16), keeping their signs
template <bool kBf16>
__device__ __forceinline__ uint32_t flush_denormals2(uint32_t u) {
    constexpr uint32_t kMinNormal = kBf16 ? 0x0080u : 0x0400u;
    const uint32_t mag = u & 0x7FFF7FFFu;
    uint32_t keep = 0x80008000u;
    if ((mag & 0xFFFFu) >= kMinNormal) keep |= 0x00007FFFu;
    if ((mag >> 16) >= kMinNormal) keep |= 0x7FFF0000u;
    return u & keep;
}

// the 16-bit code of an fp32 container that holds a value of the type (exact)
template <bool kBf16>
__device__ __forceinline__ uint32_t to_16(float v) {
    return kBf16 ? (__float_as_uint(v) >> 16) : (uint32_t)__half_as_ushort(__float2half_rn(v));
}

// master + h in fp32, h a 16-bit value: the mixed-precision add converts h exactly and rounds the sum
// once (to nearest even, denormals kept), which is what a conversion followed by an fp32 addition does,
// in one instruction.
template <bool kBf16>
__device__ __forceinline__ float add_16_to_master(float master, unsigned short h) {
    float r;
    if (kBf16) asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(r) : "h"(h), "f"(master));
    else asm("add.rn.f32.f16 %0, %1, %2;" : "=f"(r) : "h"(h), "f"(master));
    return r;
}

// The part of a 32-deep slice of an operand tile (kRows rows of op(A), or columns of op(B)) that a
// thread fetches: kRows * 32 / 1024 groups of four elements that are consecutive in memory (four k
// of a row when k is the contiguous index, four rows of a k otherwise).  A group inside the matrix
// of a 16-byte aligned operand is one 128-bit load; at the edges, and for other operands, its
// elements are loaded one by one, zero outside the matrix.
template <int kRows>
__device__ __forceinline__ void group_position(int f, int k_major, int& r, int& k) {
    if (k_major) { r = f / (kFmBK / 4); k = 4 * (f % (kFmBK / 4)); }
    else { k = f / (kRows / 4); r = 4 * (f % (kRows / 4)); }
}
template <int kRows>
__device__ __forceinline__ void fetch_slice(float4 (&v)[kRows * kFmBK / (4 * kFmThreads)], const float* src, long long ld,
                                            int k_major, int vec_ok, int r0, int rmax, int k0, int kmax) {
#pragma unroll
    for (int t = 0; t < kRows * kFmBK / (4 * kFmThreads); ++t) {
        int r, k;
        group_position<kRows>(threadIdx.x + t * kFmThreads, k_major, r, k);
        r += r0;
        k += k0;
        const float* ptr = k_major ? src + (long long)r * ld + k : src + (long long)k * ld + r;
        const bool full = k_major ? (r < rmax && k + 3 < kmax) : (k < kmax && r + 3 < rmax);
        if (vec_ok && full) {
            v[t] = *reinterpret_cast<const float4*>(ptr);
        } else {
            float e[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int rr = k_major ? r : r + j, kk = k_major ? k + j : k;
                e[j] = (rr < rmax && kk < kmax) ? (k_major ? ptr[j] : ptr[j]) : 0.0f;
            }
            v[t] = make_float4(e[0], e[1], e[2], e[3]);
        }
    }
}

template <bool kStats, bool kFlush, bool kBf16, bool kConv>
__global__ void __launch_bounds__(kFmThreads, kConv ? kHfConvBlocksPerSm : kHfBlocksPerSm)
fmac8_f16_kernel(FmacParams g, QuantParams p, qfmt_stats_t* __restrict__ stats) {
    __shared__ __align__(16) uint32_t As2[kFmBK][kHfBM + 4];  // each A value twice: {a, a} as f16x2
    __shared__ __align__(16) uint16_t Bs[kFmBK][kHfBN + 8];
    __shared__ ConvTables tabs[1];  // used by the convolution instantiations only
    extern __shared__ uint32_t lane_hist[];
    const int nbins = p.top + kExtraBins;
    const int lane = threadIdx.x & 31;
    if (kStats) {
        for (int i = threadIdx.x; i < nbins * 32; i += kFmThreads) lane_hist[i] = 0u;
        __syncthreads();
    }
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const int tiles_n = (g.N + kHfBN - 1) / kHfBN, tiles_m = (g.M + kHfBM - 1) / kHfBM;
    constexpr int kPerA = kHfBM * kFmBK / (4 * kFmThreads), kPerB = kHfBN * kFmBK / (4 * kFmThreads);  // groups of four a thread moves
    for (long long tile = blockIdx.x; tile < (long long)tiles_m * tiles_n; tile += gridDim.x) {
        const int m0 = (int)(tile / tiles_n) * kHfBM, n0 = (int)(tile % tiles_n) * kHfBN;
        float master[kHfTM][kHfTN];
        uint32_t small[kHfTM][kHfTN / 2];  // pairs of 16-bit accumulators
        const uint32_t zero2 = 0u;
#pragma unroll
        for (int i = 0; i < kHfTM; ++i) {
#pragma unroll
            for (int j = 0; j < kHfTN; ++j) master[i][j] = 0.0f;
#pragma unroll
            for (int j = 0; j < kHfTN / 2; ++j) small[i][j] = zero2;
        }
        float4 fa[kPerA], fb[kPerB];  // the next slice, on its way from global memory while this one is used
        if (kConv) {
            conv_tables<kHfBM, kHfBN>(tabs[0], g.cv, false, m0, n0, 0);  // read after the next barrier
        } else {
            fetch_slice<kHfBM>(fa, g.A, g.lda, !g.transA, g.vec_a, m0, g.M, 0, g.K);
            fetch_slice<kHfBN>(fb, g.B, g.ldb, g.transB, g.vec_b, n0, g.N, 0, g.K);
        }
        for (int k0 = 0; k0 < g.K; k0 += kFmBK) {
            __syncthreads();  // the previous slice is no longer read
            if (kConv) {  // gathered straight into the staged form
                conv_tables<kHfBM, kHfBN>(tabs[0], g.cv, true, m0, n0, k0);
                __syncthreads();
                auto twice = [](float v) { const uint32_t h = to_16<kBf16>(v); return h | (h << 16); };
                auto once = [](float v) { return (uint16_t)to_16<kBf16>(v); };
                if (g.cv.vec4) {
                    load_slice_conv4<kHfBM, kHfBM + 4, true>(As2, g, tabs[0], m0, k0, twice);
                    load_slice_conv4<kHfBN, kHfBN + 8, false>(Bs, g, tabs[0], n0, k0, once);
                } else {
                    load_slice_conv<kHfBM, kHfBM + 4, true>(As2, g, tabs[0], m0, k0, twice);
                    load_slice_conv<kHfBN, kHfBN + 8, false>(Bs, g, tabs[0], n0, k0, once);
                }
            }
            // the conversions are exact: operands hold values of the 16-bit type
#pragma unroll
            for (int t = 0; t < (kConv ? 0 : kPerA); ++t) {
                int r, k;
                group_position<kHfBM>(threadIdx.x + t * kFmThreads, !g.transA, r, k);
                const uint32_t h0 = to_16<kBf16>(fa[t].x), h1 = to_16<kBf16>(fa[t].y), h2 = to_16<kBf16>(fa[t].z),
                               h3 = to_16<kBf16>(fa[t].w);
                if (!g.transA) {  // four k of one row
                    As2[k][r] = h0 | (h0 << 16);
                    As2[k + 1][r] = h1 | (h1 << 16);
                    As2[k + 2][r] = h2 | (h2 << 16);
                    As2[k + 3][r] = h3 | (h3 << 16);
                } else {          // four rows of one k
                    *reinterpret_cast<uint4*>(&As2[k][r]) =
                        make_uint4(h0 | (h0 << 16), h1 | (h1 << 16), h2 | (h2 << 16), h3 | (h3 << 16));
                }
            }
#pragma unroll
            for (int t = 0; t < (kConv ? 0 : kPerB); ++t) {
                int r, k;
                group_position<kHfBN>(threadIdx.x + t * kFmThreads, g.transB, r, k);
                const uint32_t h0 = to_16<kBf16>(fb[t].x), h1 = to_16<kBf16>(fb[t].y), h2 = to_16<kBf16>(fb[t].z),
                               h3 = to_16<kBf16>(fb[t].w);
                if (g.transB) {   // four k of one column
                    Bs[k][r] = (uint16_t)h0;
                    Bs[k + 1][r] = (uint16_t)h1;
                    Bs[k + 2][r] = (uint16_t)h2;
                    Bs[k + 3][r] = (uint16_t)h3;
                } else {          // four columns of one k
                    *reinterpret_cast<uint2*>(&Bs[k][r]) = make_uint2(h0 | (h1 << 16), h2 | (h3 << 16));
                }
            }
            __syncthreads();
            if (!kConv && k0 + kFmBK < g.K) {
                fetch_slice<kHfBM>(fa, g.A, g.lda, !g.transA, g.vec_a, m0, g.M, k0 + kFmBK, g.K);
                fetch_slice<kHfBN>(fb, g.B, g.ldb, g.transB, g.vec_b, n0, g.N, k0 + kFmBK, g.K);
            }
            const int kmax = g.K - k0 < kFmBK ? g.K - k0 : kFmBK;
#pragma unroll 1
            for (int kg = 0; kg < kmax; kg += kGroup) {
#pragma unroll
                for (int kk = 0; kk < kGroup; ++kk) {
                    const uint4 a0 = *reinterpret_cast<const uint4*>(&As2[kg + kk][ty * kHfTM]);
                    const uint4 bv = *reinterpret_cast<const uint4*>(&Bs[kg + kk][tx * kHfTN]);  // 8 halves
                    const uint32_t aw[kHfTM] = {a0.x, a0.y, a0.z, a0.w};
                    const uint32_t bw[kHfTN / 2] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
                    for (int i = 0; i < kHfTM; ++i) {
#pragma unroll
                        for (int j = 0; j < kHfTN / 2; ++j) {
                            const uint32_t r = fma2_16<kBf16>(aw[i], bw[j], small[i][j]);
                            small[i][j] = kFlush ? flush_denormals2<kBf16>(r) : r;
                        }
                    }
                }
                // the group's sums move to the master accumulators (fp32 addition)
#pragma unroll
                for (int i = 0; i < kHfTM; ++i)
#pragma unroll
                    for (int j = 0; j < kHfTN / 2; ++j) {
                        master[i][2 * j] = add_16_to_master<kBf16>(master[i][2 * j], (unsigned short)(small[i][j] & 0xFFFFu));
                        master[i][2 * j + 1] = add_16_to_master<kBf16>(master[i][2 * j + 1], (unsigned short)(small[i][j] >> 16));
                        small[i][j] = zero2;
                    }
            }
        }
        store_patch<kStats, kHfTM, kHfTN>(g, p, master, m0 + ty * kHfTM, n0 + tx * kHfTN, lane_hist, lane);
    }
    merge_block_hist<kStats>(stats, p, lane_hist, nbins, (unsigned long long)g.M * (unsigned long long)g.N);
}

}  // namespace

// Launches the kernel for a product described by g (plain matrices, or a convolution when g.cv.mode != 0).
int launch_fmac8(const FmacParams& g, const QuantParams& p, const qfmt_format_t* fmt, qfmt_stats_t* d_stats,
                 bool use_native, bool bf16, const DeviceInfo& dev, cudaStream_t stream) {
    const bool conv = g.cv.mode != 0;
    const bool has_stats = d_stats != nullptr;
    const size_t smem = has_stats ? (size_t)(p.top + kExtraBins) * 32 * sizeof(uint32_t) : 0;
    if (use_native) {
        const long long tiles = (((long long)g.M + kHfBM - 1) / kHfBM) * (((long long)g.N + kHfBN - 1) / kHfBN);
        const long long slots = (long long)dev.sm_count * (conv ? kHfConvBlocksPerSm : kHfBlocksPerSm);
        const unsigned grid = (unsigned)(tiles < slots ? tiles : slots);
        const bool flush = fmt->denormals == 0;
        const size_t sm = has_stats ? smem : 0;
        // 256-bin histograms (bfloat16) put static + dynamic shared memory past the 48 KB that need no opt-in
#define QFMT_HLAUNCH(S, F, B, C)                                                                            \
    do {                                                                                                   \
        if (sm > 16 * 1024)                                                                                \
            QFMT_CUDA_TRY(cudaFuncSetAttribute(fmac8_f16_kernel<S, F, B, C>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm)); \
        fmac8_f16_kernel<S, F, B, C><<<grid, kFmThreads, sm, stream>>>(g, p, d_stats);                      \
    } while (0)
#define QFMT_HTYPE(S, F)                                                                                   \
    do {                                                                                                   \
        if (bf16) { if (conv) QFMT_HLAUNCH(S, F, true, true); else QFMT_HLAUNCH(S, F, true, false); }      \
        else { if (conv) QFMT_HLAUNCH(S, F, false, true); else QFMT_HLAUNCH(S, F, false, false); }         \
    } while (0)
        if (has_stats) { if (flush) QFMT_HTYPE(true, true); else QFMT_HTYPE(true, false); }
        else { if (flush) QFMT_HTYPE(false, true); else QFMT_HTYPE(false, false); }
#undef QFMT_HTYPE
#undef QFMT_HLAUNCH
    } else {
        const long long tiles = (((long long)g.M + kFmBM - 1) / kFmBM) * (((long long)g.N + kFmBN - 1) / kFmBN);
        const long long cap = (long long)dev.sm_count * kFmBlocksPerSm;
        const unsigned grid = (unsigned)(tiles < cap ? tiles : cap);
        const bool flush = fmt->denormals == 0;
        const int wide = fmt->e == 8 ? 2 : (fmt->e == 7 ? 1 : 0);
        const size_t sm = has_stats ? smem : 0;
        // 256-bin histograms (e = 8) put static + dynamic shared memory past the 48 KB that need no opt-in
#define QFMT_FLAUNCH(S, F, W)                                                                              \
    do {                                                                                                   \
        if (sm > 16 * 1024) {                                                                              \
            QFMT_CUDA_TRY(cudaFuncSetAttribute(fmac8_kernel<S, F, W, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm)); \
            QFMT_CUDA_TRY(cudaFuncSetAttribute(fmac8_kernel<S, F, W, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm)); \
        }                                                                                                  \
        if (conv) fmac8_kernel<S, F, W, true><<<grid, kFmThreads, sm, stream>>>(g, p, d_stats);             \
        else fmac8_kernel<S, F, W, false><<<grid, kFmThreads, sm, stream>>>(g, p, d_stats);                 \
    } while (0)
#define QFMT_FWIDE(S, F)                                                                                   \
    do {                                                                                                   \
        if (wide == 2) QFMT_FLAUNCH(S, F, 2); else if (wide == 1) QFMT_FLAUNCH(S, F, 1); else QFMT_FLAUNCH(S, F, 0); \
    } while (0)
        if (has_stats) { if (flush) QFMT_FWIDE(true, true); else QFMT_FWIDE(true, false); }
        else { if (flush) QFMT_FWIDE(false, true); else QFMT_FWIDE(false, false); }
#undef QFMT_FWIDE
#undef QFMT_FLAUNCH
    }
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}

int gemm_fmac8_device(const qfmt_matrix_t* A, const qfmt_matrix_t* B, float* d_C, int64_t ldc, const qfmt_format_t* fmt,
                      qfmt_stats_t* d_stats, int accumulate, int path, cudaStream_t stream) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    if (fmt->m > 10) return QFMT_ERR_BAD_FORMAT;  // operands of at most 11 significant bits
    if (A == nullptr || B == nullptr) return QFMT_ERR_BAD_ARG;
    if (accumulate != 0 && accumulate != 1) return QFMT_ERR_BAD_ARG;
    if (path < 0 || path > 2) return QFMT_ERR_BAD_ARG;
    const int64_t M = A->trans ? A->cols : A->rows, K = A->trans ? A->rows : A->cols;
    const int64_t Kb = B->trans ? B->cols : B->rows, N = B->trans ? B->rows : B->cols;
    if (M < 0 || N < 0 || K < 0 || K != Kb || M > 0x7FFFFFFF || N > 0x7FFFFFFF || K > 0x7FFFFFFF) return QFMT_ERR_BAD_ARG;
    if (A->ld < A->cols || B->ld < B->cols || ldc < N) return QFMT_ERR_BAD_ARG;
    if ((M != 0 && K != 0 && A->ptr == nullptr) || (N != 0 && K != 0 && B->ptr == nullptr) ||
        (M != 0 && N != 0 && d_C == nullptr))
        return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(A->ptr) & 3u) || (reinterpret_cast<uintptr_t>(B->ptr) & 3u) ||
        (reinterpret_cast<uintptr_t>(d_C) & 3u) || (reinterpret_cast<uintptr_t>(d_stats) & 7u))
        return QFMT_ERR_BAD_ARG;
    const bool bf16 = fmt->e == 8 && fmt->m == 7;
    const bool native = (fmt->e == 5 && fmt->m == 10) || bf16;
    if (path == 2 && !native) return QFMT_ERR_BAD_FORMAT;
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;
    if (d_stats != nullptr && accumulate == 0) QFMT_CUDA_TRY(cudaMemsetAsync(d_stats, 0, sizeof(qfmt_stats_t), stream));
    if (M == 0 || N == 0) return QFMT_OK;

    qfmt_format_t f = *fmt;
    f.loss_scale = 1.0f;  // operands are already scaled and rounded; nothing is scaled here
    const QuantParams p = make_params(f);
    FmacParams g;
    g.A = A->ptr; g.B = B->ptr; g.C = d_C;
    g.lda = A->ld; g.ldb = B->ld; g.ldc = ldc;
    g.M = (int)M; g.N = (int)N; g.K = (int)K;
    g.transA = A->trans ? 1 : 0; g.transB = B->trans ? 1 : 0;
    g.vec_store = (ldc % 4 == 0) && !(reinterpret_cast<uintptr_t>(d_C) & 15u);
    g.vec_a = (A->ld % 4 == 0) && !(reinterpret_cast<uintptr_t>(A->ptr) & 15u);
    g.vec_b = (B->ld % 4 == 0) && !(reinterpret_cast<uintptr_t>(B->ptr) & 15u);
    g.cv = ConvGather{};  // mode 0: plain matrices
    return launch_fmac8(g, p, fmt, d_stats, native && path != 1, bf16, dev, stream);
}

// The three products of a convolution with FMAC-8 accumulation, on channels-last tensors (see the
// head of this file for the order of the reduction).
int conv_fmac8_device(int op, const qfmt_conv_t* geom, const float* d_p, const float* d_q, float* d_out,
                      const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate, int path, cudaStream_t stream) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    if (fmt->m > 10) return QFMT_ERR_BAD_FORMAT;
    if (geom == nullptr || op < QFMT_CONV_FWD || op > QFMT_CONV_WGRAD) return QFMT_ERR_BAD_ARG;
    if (accumulate != 0 && accumulate != 1) return QFMT_ERR_BAD_ARG;
    if (path < 0 || path > 2) return QFMT_ERR_BAD_ARG;
    const qfmt_conv_t& c = *geom;
    if (c.n <= 0 || c.c_in <= 0 || c.h <= 0 || c.w <= 0 || c.c_out <= 0 || c.r <= 0 || c.s <= 0 || c.pad_h < 0 || c.pad_w < 0)
        return QFMT_ERR_BAD_ARG;
    const int64_t oh = (int64_t)c.h + 2 * c.pad_h - c.r + 1, ow = (int64_t)c.w + 2 * c.pad_w - c.s + 1;
    if (oh <= 0 || ow <= 0) return QFMT_ERR_BAD_ARG;
    const int64_t taps = (int64_t)c.r * c.s, in_px = (int64_t)c.n * c.h * c.w, out_px = (int64_t)c.n * oh * ow;
    // every tensor, and every index the kernel forms, stays below 2^31
    const int64_t lim = 0x7FFFFFFF;
    if (in_px * c.c_in > lim || out_px * c.c_out > lim || taps * c.c_in * c.c_out > lim ||
        (taps + 32) * ((int64_t)c.c_in + c.c_out) > lim || in_px + 64 > lim || out_px + 64 > lim)
        return QFMT_ERR_BAD_ARG;
    if (d_p == nullptr || d_q == nullptr || d_out == nullptr) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_p) & 3u) || (reinterpret_cast<uintptr_t>(d_q) & 3u) ||
        (reinterpret_cast<uintptr_t>(d_out) & 3u) || (reinterpret_cast<uintptr_t>(d_stats) & 7u))
        return QFMT_ERR_BAD_ARG;
    const bool bf16 = fmt->e == 8 && fmt->m == 7;
    const bool native = (fmt->e == 5 && fmt->m == 10) || bf16;
    if (path == 2 && !native) return QFMT_ERR_BAD_FORMAT;
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;
    if (d_stats != nullptr && accumulate == 0) QFMT_CUDA_TRY(cudaMemsetAsync(d_stats, 0, sizeof(qfmt_stats_t), stream));

    qfmt_format_t f = *fmt;
    f.loss_scale = 1.0f;
    const QuantParams p = make_params(f);
    FmacParams g;
    g.A = d_p; g.B = d_q; g.C = d_out;
    g.transA = 0; g.transB = 0; g.vec_a = g.vec_b = 0;
    ConvGather& cv = g.cv;
    cv.S = c.s; cv.taps = (int)taps;
    cv.filt_n = c.c_in; cv.filt_k = c.c_out;
    if (op == QFMT_CONV_FWD) {          // Y[pixel][c_out] = sum over (tap, c_in) of X gathered . W[c_out][(tap, c_in)]
        cv.mode = 1;
        cv.H = c.h; cv.W = c.w; cv.C = c.c_in; cv.PH = (int)oh; cv.PW = (int)ow; cv.pixels = (int)out_px;
        cv.sign = 1; cv.off_h = -c.pad_h; cv.off_w = -c.pad_w;
        g.M = (int)out_px; g.N = c.c_out; g.K = (int)(taps * c.c_in);
        g.lda = 0; g.ldb = g.K; g.ldc = c.c_out;
    } else if (op == QFMT_CONV_DGRAD) { // dX[pixel][c_in] = sum over (tap, c_out) of dY gathered . W[c_out][tap][c_in]
        cv.mode = 2;
        cv.H = (int)oh; cv.W = (int)ow; cv.C = c.c_out; cv.PH = c.h; cv.PW = c.w; cv.pixels = (int)in_px;
        cv.sign = -1; cv.off_h = c.pad_h; cv.off_w = c.pad_w;
        g.M = (int)in_px; g.N = c.c_in; g.K = (int)(taps * c.c_out);
        g.lda = 0; g.ldb = 0; g.ldc = c.c_in;
    } else {                            // dW[c_out][(tap, c_in)] = sum over output pixels of dY[pixel][c_out] . X gathered
        cv.mode = 3;
        cv.H = c.h; cv.W = c.w; cv.C = c.c_in; cv.PH = (int)oh; cv.PW = (int)ow; cv.pixels = (int)out_px;
        cv.sign = 1; cv.off_h = -c.pad_h; cv.off_w = -c.pad_w;
        g.M = c.c_out; g.N = (int)(taps * c.c_in); g.K = (int)out_px;
        g.lda = c.c_out; g.ldb = 0; g.ldc = g.N;
    }
    g.vec_store = (g.ldc % 4 == 0) && !(reinterpret_cast<uintptr_t>(d_out) & 15u);
    cv.vec4 = (c.c_in % 4 == 0 && c.c_out % 4 == 0 &&
               !((reinterpret_cast<uintptr_t>(d_p) | reinterpret_cast<uintptr_t>(d_q)) & 15u)) ? 1 : 0;
    return launch_fmac8(g, p, fmt, d_stats, native && path != 1, bf16, dev, stream);
}

}  // namespace qfmt

extern "C" int qfmt_gemm_fmac8(const qfmt_matrix_t* A, const qfmt_matrix_t* B, float* d_C, int64_t ldc,
                               const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate, int path, void* stream) {
    return qfmt::gemm_fmac8_device(A, B, d_C, ldc, fmt, d_stats, accumulate, path, (cudaStream_t)stream);
}

extern "C" int qfmt_conv_fmac8(int32_t op, const qfmt_conv_t* geom, const float* d_p, const float* d_q, float* d_out,
                               const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate, int path, void* stream) {
    return qfmt::conv_fmac8_device(op, geom, d_p, d_q, d_out, fmt, d_stats, accumulate, path, (cudaStream_t)stream);
}
