// Contraction of format-rounded operands with fp32 accumulation on the tcgen05 tensor cores.
//
// Semantics: the FMACS instruction of Section III-B, a32 = round(a32 + x16 * y16): products of
// 16-bit-format values are formed exactly and accumulated in fp32.  Every value of a 1/e/m
// format with e <= 8 and m <= 10 is exactly a TF32 number (8 exponent bits, 10 mantissa bits),
// so kind::tf32 MMAs multiply the operands exactly and only the order of the fp32 accumulation
// differs from any other FMACS evaluation.
//
// Kernel: persistent, one CTA per SM, warp specialised.
//   warp 0      TMA producer: fills a ring of kStages shared-memory stages, each holding a
//               128 x 32 tile of op(A) and a 256 x 32 tile of op(B) in the 128-byte-swizzled
//               layout the MMA descriptors expect (K-major operands: one box per operand;
//               MN-major operands: one 32 x 32 box per 32 rows/columns of the tile).
//   warp 1      MMA issuer: one thread issues four 128x256x8 tcgen05.mma per stage into one of
//               two 256-column TMEM accumulators and commits to the stage's "empty" barrier.
//   warps 2-3   idle (they complete the first warpgroup, which gives most of its registers away)
//   warps 4-11  accumulate + epilogue: see "two-level summation" below.
//
// Two-level summation.  The tensor core adds each MMA's eight products to the fp32 accumulator
// and truncates (rounds toward zero) once per MMA, so one long TMEM accumulation drifts by about
// (K/8) * 2^-24 relative to sum |a||b| (measured: 2^-14 at K = 8192 with same-sign data).  The
// kernel therefore accumulates only kChunkK = 64 consecutive K elements (eight MMAs) per TMEM
// accumulator, starting each chunk from zero, and the eight accumulate warps add the finished
// chunk sums, in K order, to a running sum in registers with round-to-nearest-even adds while
// the MMA warp fills the other TMEM accumulator.  Each warp owns TMEM lane quadrant warp_id % 4
// and one 128-column half of the tile: 128 running sums per thread.
// A third level keeps the sequential part short: after kFlushChunks chunk sums (1024 K elements)
// the register sums are added into the C tile itself and reset, so an output sees at most
// kFlushChunks + K/1024 rounded additions of large partial sums instead of K/64.
//
// Packed 16-bit operands.  1/5/10 codes are IEEE binary16 words and 1/8/7 codes are bfloat16 words,
// so for these two formats the CTA-pair kernel (gemm_tf32_pair_kernel, despite its name) is also
// instantiated with kind::f16 MMAs that read the codes as they are stored: a stage is then 64 K
// elements per 128-byte row, a chunk 128 K elements (still eight MMAs) and a group 2048; the
// products are as exact as in TF32 and the three levels are the same (gemm16_device).
//
// Every mbarrier wait is bounded; on expiry the thread records QFMT_ERR_TIMEOUT in the status
// word, raises a CTA-wide abort flag and every role drains to the common exit, where TMEM is
// released.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "common.cuh"
#include "ptx.cuh"
#include "round.cuh"

namespace qfmt {
namespace {

constexpr int kBM = 128;            // tile rows (MMA M)
constexpr int kBN = 256;            // tile columns (MMA N)
constexpr int kBK = 32;             // K elements per stage: 128 bytes, one swizzle row
constexpr int kMmaK = 8;            // K per tcgen05.mma of kind::tf32
constexpr int kStages = 3;
constexpr int kAccCols = kBN;       // TMEM columns per accumulator
constexpr int kTmemCols = 512;      // two accumulators
constexpr int kThreads = 384;         // warpgroup 0: producer + MMA warps; warpgroups 1-2: accumulate warps
constexpr int kChunkKB = 2;           // stages per TMEM accumulation: 64 K elements, 8 MMAs
constexpr int kAccWarps = 8;
constexpr int kFlushChunks = 16;       // chunk sums per level-1 group before the running sums move to C
constexpr uint32_t kABytes = kBM * kBK * 4;
constexpr uint32_t kBBytes = kBN * kBK * 4;
constexpr uint32_t kStageBytes = kABytes + kBBytes;
// Output staging: each accumulate warp moves its 32 x 128 block to C in four passes of 32 columns
// through two alternating 32 x 32 boxes (rows of 128 bytes, 16-byte chunks XOR-swizzled with the
// row index: conflict-free for the row-per-lane writes and the layout a 128B-swizzled TMA store
// reads).  While one box is being read by its copy the other is filled.
constexpr int kOutCols = 32;
constexpr uint32_t kOutBoxBytes = 32 * 32 * 4;
constexpr uint32_t kOutWarpBytes = 2 * kOutBoxBytes;
constexpr uint32_t kOutBytes = kAccWarps * kOutWarpBytes;
// Layer-output epilogue (Y = R(R(acc) + R(B)) with statistics): one counter per bin for the CTA.
constexpr int kEpiBins = 128;  // 2^6 - 1 + the split bins, rounded up (formats with e <= 6)
constexpr uint32_t kEpiHistBytes = kEpiBins * 4;
constexpr uint32_t kSmemBytes = kStages * kStageBytes + kOutBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kEpiHistBytes;
constexpr uint32_t kWaitLimit = 1u << 31;  // SM cycles (about a second) before a wait is declared dead

struct GemmParams {
    int M, N, K;
    long long ldc;
    float* C;
    // Status area at the head of the workspace: two 64-bit words.  Word 1 receives the launch's tag when
    // the kernel starts; an error is recorded in word 0 as (tag << 16) | code.  A reader takes word 0 for
    // an error only if its tag is word 1's, so nothing has to be cleared before a launch and whatever an
    // earlier call (or nobody) left there reads as "no error".
    unsigned long long* status;
    unsigned long long launch_tag;
    int a_mn_major;  // op(A) stored with M contiguous
    int b_mn_major;  // op(B) stored with N contiguous
    int tiles_m, tiles_n;
    int tma_store;   // C base, row pitch and row length are multiples of 16 bytes: C is written by TMA
    int c_blocked;   // pair kernel: N is a multiple of 32 and the C map is {32, rows, N / 32, splits}
    // Balanced schedule (mode 1 only, sk_cpt > 0).  The tiles' 64-element K chunks form one sequence,
    // tile after tile, and CTA b works on the b-th of gridDim.x equal ranges of it: up to sk_pieces
    // consecutive tiles, the first and the last possibly in part.  A piece that begins inside a tile
    // writes to the CTA's slot in sk_partials ([gridDim.x][tile_rows][N]) instead of C; a later
    // kernel adds the slot to C.  Ranges are at least a tile long, so no tile has two such pieces.
    int sk_cpt;              // chunks per tile, 0 = schedule off
    int sk_pieces;           // pieces a CTA may have
    float* sk_partials;
    // The same schedule in the pair kernel (sk_flags != nullptr), dealt among the CTA pairs, without the
    // slots and without the second kernel.  A pair runs the piece that begins inside a tile LAST and adds
    // it into C at the destination; by then the pair before it, whose range ends inside that tile, has
    // written the tile's first part as the FIRST piece of its own range and has said so in
    // sk_flags (one word per pair, 64 bytes apart, zeroed before the launch).  A tile has at most two pieces
    // (ranges are at least a tile long), the first stored and the second added after it in program
    // order of a flag hand-over, so the sums are the same on every run.
    int* sk_flags;
    int sk_q, sk_r;          // quotient and remainder of (tiles * sk_cpt) / pairs
    int wg_padded;   // filter gradient, padded stages: an image row takes a power-of-two number of K rows
                     // (the copy engine zero-fills the columns past the image), a stage is 32 K rows
                     // exactly, and one rank-5 copy per operand brings all of its channel blocks
    int rows_box;    // filter gradient: image rows fetched by one copy (rows_per_blk when it divides the image height, else 1)
    int wg_segs;     // filter gradient: K stages per output row (1; more when a row is longer than a stage's 32 pixels)
    int a_blocked, b_blocked;  // dense MN-major operand whose extent is a multiple of 32: its map is
                               // rank 3, {32, K, extent / 32}, and one copy fetches a stage's 32-wide blocks
    // ---- work decomposition
    int tile_rows;         // rows of C owned by one M-tile (128, or whole image rows in mode 1)
    int kb_total;          // stages (k-blocks) in the whole contraction
    int kb_per_split;      // stages handled by one work item
    int splits;            // split-K factor; the partial result of split s goes to C + s * split_stride
    long long split_stride;
    uint32_t a_bytes, b_bytes;  // bytes TMA delivers per stage
    // ---- convolution modes (see conv_device): 0 dense, 1 pixels are the M dimension (forward and
    // data gradient), 2 pixels are the K dimension (filter gradient)
    int mode;
    int img_rows, img_w;   // rows per image and pixels per row of the pixel space that is tiled
    int total_q;           // batch * img_rows
    int rows_per_blk;      // image rows per M-tile (mode 1) or per stage (mode 2)
    int taps, taps_s;      // R*S and S
    int cblocks, ck;       // mode 1: 32-channel blocks per tap and contraction channels; mode 2: ck = C_in
    int tap_sign, off_h, off_w;  // activation row read for tap (r, s): h + tap_sign * r + off_h
    int full_tiles_m;      // mode 1: M-tiles that are complete (the C tensor map covers exactly these)
    int conv_rows;         // mode 1 on CTA pairs: pixels (rows of C) in one CTA's M-tile
    // ---- layer-output epilogue (dense mode, one summation group, no split K): the sums are rounded,
    // the rounded bias of their column is added, the result is rounded again and counted, all in the
    // accumulate warps' registers before the tile is stored
    int epi;                  // 0 = off
    const float* epi_rbias;   // rounded bias, padded with zeros to tiles_n * kBN entries
    qfmt_stats_t* epi_stats;  // may be null
    QuantParams epi_q;
};

// Mode 1 reads the pixel operand through maps whose boxes hold 1 .. kMaxRowMaps whole image rows
// (32 channels x img_w pixels x cnt rows), so that a tile's rows are fetched with one box per
// image they touch instead of one box per row.
constexpr int kMaxRowMaps = 16;
struct RowMaps {
    CUtensorMap m[kMaxRowMaps];
};

// Position of work item t: tile coordinates, split, and the range of stages it sums.
struct WorkItem {
    int tile_m, tile_n, split, m0, n0, kb_begin, num_kb;
    int partial;  // balanced schedule: the piece begins inside its tile and goes to the CTA's slot
    int head;     // balanced schedule of the pair kernel: the next pair adds the rest of this tile
};
// Piece j (in the order a pair runs them) of pair `unit` under the balanced schedule of the pair
// kernel: first the range's last piece if it ends before its tile does (`head`: the next pair finishes
// that tile, and needs it stored early), then the whole tiles in their natural order, last the range's
// first piece if it begins inside a tile (`partial`: it adds to what the pair before has stored).
// Every pair starts at the same moment and ranges are at least a tile long, so a head piece (at most a
// tile) is in C before the pair after it has worked through the rest of its range and the first
// summation group of its partial piece.
struct PairPiece {
    int tile, kb_begin, num_kb, partial, head;
};
// Range boundaries come from the quotient q and remainder r of total / units, so that everything
// stays in 32 bits: lo(u) = q * u + r * u / units (total < 2^31, units < 2^15).
__host__ __device__ __forceinline__ PairPiece pair_piece(int q, int r, int cpt, int kb_total, int units, int unit, int j) {
    PairPiece pc = {0, 0, 0, 0, 0};
    const int lo = q * unit + r * unit / units, hi = q * (unit + 1) + r * (unit + 1) / units;
    if (hi <= lo) return pc;
    const int first_tile = lo / cpt, last_tile = (hi - 1) / cpt;
    const int n_nat = last_tile - first_tile + 1;
    const bool first_partial = lo > first_tile * cpt, last_head = hi < (last_tile + 1) * cpt;
    int nat;
    if (last_head && j == 0) {
        nat = n_nat - 1;
    } else {
        const int idx = last_head ? j - 1 : j, m = last_head ? n_nat - 1 : n_nat;  // the other pieces
        if (idx >= m) return pc;
        nat = first_partial ? (idx + 1 < m ? idx + 1 : 0) : idx;
    }
    const int tile = first_tile + nat, first = tile * cpt;
    const int s = lo > first ? lo : first, e = hi < first + cpt ? hi : first + cpt;
    pc.tile = tile;
    pc.kb_begin = (s - first) * kChunkKB;
    const int kb_end = (e - first) * kChunkKB < kb_total ? (e - first) * kChunkKB : kb_total;
    pc.num_kb = kb_end - pc.kb_begin;
    pc.partial = s > first ? 1 : 0;
    pc.head = e < first + cpt ? 1 : 0;
    return pc;
}

// Chunk range [lo, hi) of CTA b under the balanced schedule.
__host__ __device__ __forceinline__ void sk_range(long long total, int ctas, int b, long long* lo, long long* hi) {
    *lo = total * b / ctas;
    *hi = total * (b + 1) / ctas;
}
__device__ __forceinline__ WorkItem decode_work(const GemmParams& p, int t) {
    WorkItem w;
    const int num_tiles = p.tiles_m * p.tiles_n;
    w.partial = 0;
    w.head = 0;
    if (p.sk_cpt > 0) {
        // t = b + piece * gridDim.x for CTA b
        const int ctas = (int)gridDim.x, b = t % ctas, piece = t / ctas;
        long long lo, hi;
        sk_range((long long)num_tiles * p.sk_cpt, ctas, b, &lo, &hi);
        const long long tile = lo / p.sk_cpt + piece, first = tile * p.sk_cpt;
        const long long s = lo > first ? lo : first, e = hi < first + p.sk_cpt ? hi : first + p.sk_cpt;
        w.split = 0;
        if (s >= e) {  // no such piece
            w.tile_m = w.tile_n = w.m0 = w.n0 = w.kb_begin = w.num_kb = 0;
            return w;
        }
        w.tile_m = (int)(tile % p.tiles_m);
        w.tile_n = (int)(tile / p.tiles_m);
        w.m0 = w.tile_m * p.tile_rows;
        w.n0 = w.tile_n * kBN;
        w.kb_begin = (int)(s - first) * kChunkKB;
        const int kb_end = (int)(e - first) * kChunkKB < p.kb_total ? (int)(e - first) * kChunkKB : p.kb_total;
        w.num_kb = kb_end - w.kb_begin;
        w.partial = s > first ? 1 : 0;
        return w;
    }
    const int tile = t % num_tiles;
    w.split = t / num_tiles;
    w.tile_m = tile % p.tiles_m;
    w.tile_n = tile / p.tiles_m;
    w.m0 = w.tile_m * p.tile_rows;
    w.n0 = w.tile_n * kBN;
    w.kb_begin = w.split * p.kb_per_split;
    const int kb_end = w.kb_begin + p.kb_per_split < p.kb_total ? w.kb_begin + p.kb_per_split : p.kb_total;
    w.num_kb = kb_end - w.kb_begin;
    return w;
}

// Shared-memory matrix descriptor.  Addresses and offsets are stored in 16-byte units.
//   K-major tile (layout 2, 128-byte swizzle of 16-byte chunks): rows of 128 bytes (32 K
//       elements), 8-row groups 1024 bytes apart (stride offset); leading offset unused.
//   MN-major tile (layout 1, 128-byte swizzle of 32-byte chunks: the one layout 32-bit
//       operands may use when M/N is the contiguous dimension): blocks of [32 K-rows][128
//       bytes = 32 M/N elements]; leading offset = distance between blocks, stride offset =
//       distance between groups of 4 K-rows (512 bytes).
constexpr uint32_t kLayoutSw128 = 2, kLayoutSw128Base32 = 1;
// Field positions: start address bits 0-13, leading offset bits 16-29, stride offset bits 32-45,
// descriptor version (1 on sm_100) bits 46-47, layout bits 61-63.  The descriptor is kept as a
// constant high word and a low word to which the tile's offset (in 16-byte units) is added, so
// that the MMA thread spends one add per operand per MMA.
__device__ __forceinline__ uint32_t desc_hi(uint32_t sbo_bytes, uint32_t layout) {
    return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (layout << 29);
}
__device__ __forceinline__ uint32_t desc_lo(uint32_t saddr, uint32_t lbo_bytes) {
    return ((saddr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__device__ __forceinline__ uint64_t desc_join(uint32_t hi, uint32_t lo) {
    return ((uint64_t)hi << 32) | lo;
}

__device__ __forceinline__ uint32_t make_idesc(int a_mn, int b_mn) {
    return (1u << 4)                     // D format: fp32
           | (2u << 7) | (2u << 10)      // A, B format: TF32
           | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16)
           | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

// What a role does when one of its bounded waits runs out: the CTA-wide flag tells the other roles
// to stop at their next check, the status area (first error of the launch wins) tells the host.
__device__ __forceinline__ void raise_timeout(unsigned long long* status, unsigned long long tag, volatile int* abort_flag) {
    *abort_flag = 1;
    const unsigned long long seen = *reinterpret_cast<volatile unsigned long long*>(status);
    if ((seen >> 16) != tag)  // no error of this launch yet; if another role gets in first, its error stands
        atomicCAS(status, seen, (tag << 16) | (unsigned long long)(-(int)QFMT_ERR_TIMEOUT));
}
__device__ __forceinline__ void raise_timeout(const GemmParams& p, volatile int* abort_flag) {
    raise_timeout(p.status, p.launch_tag, abort_flag);
}
// The first thread of the grid names the launch in the status area (see GemmParams::status).
__device__ __forceinline__ void announce_launch(unsigned long long* status, unsigned long long tag) {
    if (blockIdx.x == 0 && threadIdx.x == 0) *reinterpret_cast<volatile unsigned long long*>(status + 1) = tag;
}

// Self-test of the bounded-wait path with the primitives the GEMM kernels use, on a barrier that
// nothing ever arrives on.  Warp 0 plays a role whose wait runs out after `limit` cycles: it must
// come back from mbar_wait_bounded with false and raise the timeout.  Warp 1 plays a role that is
// not itself stuck: it polls the abort flag (itself bounded, at 64 limits) and leaves when the flag
// is up.  Both meet at the common exit and the kernel returns normally; nothing can spin forever.
// trace[0] = 1 if warp 0's wait returned false, trace[1] = 1 if warp 1 left because of the flag,
// trace[2] = cycles warp 0 waited.
__global__ void __launch_bounds__(64, 1)
bounded_wait_selftest_kernel(unsigned long long* status, unsigned long long tag, uint32_t limit, int* trace) {
    announce_launch(status, tag);
    __shared__ __align__(8) unsigned long long bar_storage;
    __shared__ int abort_word;
    volatile int* abort_flag = &abort_word;
    const uint32_t bar = ptx::smem_addr(&bar_storage);
    if (threadIdx.x == 0) {
        ptx::mbar_init(bar, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) {
        if (lane == 0) {
            const long long t0 = clock64();
            const bool ok = ptx::mbar_wait_bounded(bar, 0u, limit);  // phase 0 never completes
            trace[2] = (int)(clock64() - t0);
            if (!ok) {
                raise_timeout(status, tag, abort_flag);
                trace[0] = 1;
            }
        }
        __syncwarp();
    } else {
        if (lane == 0) {
            const long long t0 = clock64();
            int saw = 0;
            while (clock64() - t0 < 64ll * (long long)limit) {
                if (*abort_flag) { saw = 1; break; }
                __nanosleep(64);
            }
            trace[1] = saw;
        }
        __syncwarp();
    }
    __syncthreads();
}

// Layer-output epilogue on one thread's 128 sums of a row (columns col_base + 0..127; sum2[i] holds
// columns 2i and 2i+1): Y = R(R(acc) + R(B)) of Section IV-A's worked example, then one count per
// element.  The warp counts in its own output staging boxes, idle at this point, used as a
// histogram of [128 bins][16 slots] (a lane adds to slot lane mod 16, so at most two lanes share a
// counter); afterwards the slots are summed into the CTA's histogram.  Needs at most 128 bins
// (e <= 6).
__device__ __forceinline__ void epi_transform(unsigned long long (&sum2)[64], const GemmParams& p, bool row_ok,
                                              int col_base, uint32_t* warp_hist, uint32_t* hist, int lane) {
    const uint32_t inf_bits = (uint32_t)(p.epi_q.top + p.epi_q.code_off) << 23;
    const bool count = p.epi_stats != nullptr;
    if (count) {
        if (lane == 0) ptx::bulk_wait_read_all();  // copies of the previous tile no longer read the boxes
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 64; ++i) warp_hist[i * 32 + lane] = 0u;
        __syncwarp();
    }
    const int slot = lane & 15;
#pragma unroll  // fully: sum2 must stay in registers
    for (int i = 0; i < 64; ++i) {
        const int col = col_base + 2 * i;
        const float2 rb = *reinterpret_cast<const float2*>(p.epi_rbias + col);  // same address for the whole warp
        const float2 v = ptx::unpack2(sum2[i]);
        int b0, b1;
        const uint32_t r0 = round_value<false>(__float_as_uint(v.x), p.epi_q, inf_bits);
        const uint32_t r1 = round_value<false>(__float_as_uint(v.y), p.epi_q, inf_bits);
        const uint32_t q0 = round_sum(__float_as_uint(add_ieee(__uint_as_float(r0), rb.x)), p.epi_q, b0);
        const uint32_t q1 = round_sum(__float_as_uint(add_ieee(__uint_as_float(r1), rb.y)), p.epi_q, b1);
        sum2[i] = ptx::pack2(__uint_as_float(q0), __uint_as_float(q1));
        if (count && row_ok) {
            if (col < p.N) atomicAdd(&warp_hist[b0 * 16 + slot], 1u);
            if (col + 1 < p.N) atomicAdd(&warp_hist[b1 * 16 + slot], 1u);
        }
    }
    if (count) {
        __syncwarp();
        const int nbins = p.epi_q.top + kExtraBins;
        for (int b = lane; b < nbins; b += 32) {
            uint32_t c = 0u;
#pragma unroll
            for (int s = 0; s < 16; ++s) c += warp_hist[b * 16 + ((s + lane) & 15)];
            if (c != 0u) atomicAdd(&hist[b], c);
        }
        __syncwarp();  // the boxes are about to be refilled with the tile's values
    }
}

// Folds the CTA's epilogue histogram into the device record (all threads of the CTA call it).
__device__ __forceinline__ void epi_merge(const GemmParams& p, const uint32_t* hist) {
    if (!p.epi || p.epi_stats == nullptr) return;
    const int nbins = p.epi_q.top + kExtraBins;
    for (int b = 1 + (int)threadIdx.x; b < nbins; b += kThreads) {
        const uint32_t c = hist[b];
        if (c != 0u) merge_bin(p.epi_stats, p.epi_q, b, c);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0)
        atomicAdd((unsigned long long*)&p.epi_stats->n_total, (unsigned long long)p.M * (unsigned long long)p.N);
}

// kEpi: the layer-output epilogue is compiled in (its own instantiation, so that plain products
// carry none of its code)
template <bool kEpi>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tf32_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_c, const __grid_constant__ CUtensorMap tmap_p,
                 const __grid_constant__ RowMaps row_maps, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_addr(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
    const uint32_t out_stage = tiles + kStages * kStageBytes;
    const uint32_t bars = out_stage + kOutBytes;
    // barrier layout (8 bytes each): full[kStages], empty[kStages], acc_full[2], acc_empty[2]; then
    // the TMEM base address and the abort flag.
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kStages + s); };
    auto acc_full_bar = [&](int a) { return bars + 8u * (2 * kStages + a); };
    auto acc_empty_bar = [&](int a) { return bars + 8u * (2 * kStages + 2 + a); };
    uint8_t* gen_bars = smem_raw + (bars - raw);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_bars + 8 * (2 * kStages + 4));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_bars + 8 * (2 * kStages + 4) + 8);
    // issue_progress[i]: chunks (counted over the whole kernel) up to which MMA issuer i has seen its operands arrive
    volatile uint32_t* issue_progress = reinterpret_cast<volatile uint32_t*>(gen_bars + 8 * (2 * kStages + 4) + 16);
    uint32_t* epi_hist = reinterpret_cast<uint32_t*>(gen_bars + 256);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    if (kEpi) {
        for (int i = threadIdx.x; i < kEpiBins; i += kThreads) epi_hist[i] = 0u;
    }

    if (p.mode == 2) {
        // Filter gradient: a stage holds fewer than 32 pixel rows of K; the rows TMA never writes
        // must read as zero in both operands.
        float4* z = reinterpret_cast<float4*>(smem_raw + (tiles - raw));
        for (uint32_t i = threadIdx.x; i < kStages * kStageBytes / 16; i += kThreads) z[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        ptx::fence_proxy_async();
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(acc_full_bar(a), 1);
            ptx::mbar_init(acc_empty_bar(a), kAccWarps);  // one arrival per accumulate warp
        }
        *abort_flag = 0;
        issue_progress[0] = 0;
        issue_progress[1] = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_a);
        ptx::prefetch_tensormap(&tmap_b);
        if (p.tma_store) ptx::prefetch_tensormap(&tmap_c);
        if (p.sk_cpt > 0) ptx::prefetch_tensormap(&tmap_p);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
        ptx::tmem_relinquish();
    }
    // Everything above touched shared and tensor memory only and may run while the kernel before this one
    // in the stream drains; from here on global memory is read and written.
    grid_dependency_wait();
    announce_launch(p.status, p.launch_tag);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    grid_launch_dependents();
    const uint32_t tmem_base = *tmem_slot;

    const int num_work = p.sk_cpt > 0 ? p.sk_pieces * (int)gridDim.x : p.tiles_m * p.tiles_n * p.splits;

    // Registers are allocated per group of four warps: the producer/MMA group keeps 64 per thread,
    // the accumulate groups take 224 (128 running sums + 32 freshly loaded values + addressing).
    if (warp < 4) {
    ptx::setmaxnreg_dec<80>();
    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (p.mode != 2) {
            // Dense operands and the forward / data-gradient convolutions need one to twelve boxes per
            // stage: a single thread issues them.
            if (lane == 0) {
                int stage = 0;
                uint32_t phase = 0;
                for (int t = blockIdx.x; t < num_work && !*abort_flag; t += gridDim.x) {
                    const WorkItem w = decode_work(p, t);
                    for (int kb = w.kb_begin; kb < w.kb_begin + w.num_kb; ++kb) {
                        if (!ptx::mbar_wait_bounded(empty_bar(stage), phase ^ 1u, kWaitLimit)) {
                            raise_timeout(p, abort_flag);
                            break;
                        }
                        const uint32_t sa = tiles + stage * kStageBytes;
                        const uint32_t sb = sa + kABytes;
                        const uint32_t bar = full_bar(stage);
                        ptx::mbar_expect_tx(bar, p.a_bytes + p.b_bytes);
                        if (p.mode == 0) {
                            const int k0 = kb * kBK;
                            if (p.a_blocked) {
                                ptx::tma_load_3d(sa, &tmap_a, bar, 0, k0, w.m0 >> 5);
                            } else if (p.a_mn_major) {
                                for (int c = 0; c < kBM / 32; ++c)
                                    ptx::tma_load_2d(sa + c * 4096u, &tmap_a, bar, w.m0 + c * 32, k0);
                            } else {
                                ptx::tma_load_2d(sa, &tmap_a, bar, k0, w.m0);
                            }
                            if (p.b_blocked) {
                                ptx::tma_load_3d(sb, &tmap_b, bar, 0, k0, w.n0 >> 5);
                            } else if (p.b_mn_major) {
                                for (int c = 0; c < kBN / 32; ++c)
                                    ptx::tma_load_2d(sb + c * 4096u, &tmap_b, bar, w.n0 + c * 32, k0);
                            } else {
                                ptx::tma_load_2d(sb, &tmap_b, bar, k0, w.n0);
                            }
                        } else {
                            // A: the tile's image rows at this tap's offset, one box per image touched
                            // (rows and columns outside the image read as zero: that is the padding).
                            const int tap = kb / p.cblocks, cb = kb % p.cblocks;
                            const int dh = p.tap_sign * (tap / p.taps_s) + p.off_h;
                            const int dw = p.tap_sign * (tap % p.taps_s) + p.off_w;
                            int j = 0;
                            while (j < p.rows_per_blk) {
                                const int q = w.tile_m * p.rows_per_blk + j;
                                const int h = q % p.img_rows, img = q / p.img_rows;
                                int cnt = p.rows_per_blk - j;
                                if (cnt > p.img_rows - h) cnt = p.img_rows - h;
                                if (cnt > kMaxRowMaps) cnt = kMaxRowMaps;
                                ptx::tma_load_4d(sa + (uint32_t)(j * p.img_w) * 128u, &row_maps.m[cnt - 1], bar, cb * 32, dw,
                                                 h + dh, img);
                                j += cnt;
                            }
                            if (p.b_mn_major) {  // data gradient: filters [C_out][tap][C_in] seen as
                                                 // {32, tap, C_out, C_in / 32}: one copy brings the eight column blocks
                                ptx::tma_load_4d(sb, &tmap_b, bar, 0, tap, cb * 32, w.n0 >> 5);
                            } else {             // forward: filters [C_out][tap * C_in], K contiguous
                                ptx::tma_load_2d(sb, &tmap_b, bar, tap * p.ck + cb * 32, w.n0);
                            }
                        }
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        } else {
        // The filter gradient needs 24 or more small boxes per stage: lane 0 waits for the stage and
        // arms its barrier, then the lanes issue the boxes in parallel.
        {
            int stage = 0;
            uint32_t phase = 0;
            bool dead = false;
            for (int t = blockIdx.x; t < num_work && !dead; t += gridDim.x) {
                const WorkItem w = decode_work(p, t);
                const int m0 = w.m0, n0 = w.n0;
                for (int kb = w.kb_begin; kb < w.kb_begin + w.num_kb; ++kb) {
                    const uint32_t bar = full_bar(stage);
                    int ok = 1;
                    if (lane == 0) {
                        if (!ptx::mbar_wait_bounded(empty_bar(stage), phase ^ 1u, kWaitLimit)) {
                            raise_timeout(p, abort_flag);
                            ok = 0;
                        } else if (*abort_flag) {
                            ok = 0;
                        } else {
                            ptx::mbar_expect_tx(bar, p.a_bytes + p.b_bytes);
                        }
                    }
                    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                    if (!ok) { dead = true; break; }
                    const uint32_t sa = tiles + stage * kStageBytes;
                    const uint32_t sb = sa + kABytes;
                    if (p.wg_padded) {
                        // Both operands as {32 channels, padded row, rows, image, channel block}: the
                        // tile's 256 columns lie within one tap here, so B is one box at that tap's offset.
                        if (lane == 0) {
                            const int q = kb * p.rows_per_blk;
                            const int oh = q % p.img_rows, img = q / p.img_rows;
                            const int tap = n0 / p.ck, ci = n0 % p.ck;
                            ptx::tma_load_5d(sa, &tmap_a, bar, 0, 0, oh, img, m0 >> 5);
                            ptx::tma_load_5d(sb, &tmap_b, bar, 0, tap % p.taps_s + p.off_w, oh + tap / p.taps_s + p.off_h,
                                             img, ci >> 5);
                        }
                    } else {
                        // Filter gradient: K = pixels.  A = output gradient (C_out is M), B = activations
                        // read at the tap that the N column block belongs to (C_in within a tap is N).
                        const int per_row = kBM / 32 + kBN / 32;
                        // A row longer than 32 pixels takes wg_segs stages of 32 pixels each (one image row per
                        // stage then); the last one reaches past the row's end, where the copy of A fills zeros.
                        const int x0 = (kb % p.wg_segs) * kBK, q0 = (kb / p.wg_segs) * p.rows_per_blk;
                        for (int i = lane; i < (p.rows_per_blk / p.rows_box) * per_row; i += 32) {
                            const int j = (i / per_row) * p.rows_box, c = i % per_row;
                            const int q = q0 + j;
                            const int oh = q % p.img_rows, img = q / p.img_rows;
                            const uint32_t row_off = (uint32_t)(j * p.img_w) * 128u;
                            if (c < kBM / 32) {
                                ptx::tma_load_4d(sa + c * 4096u + row_off, &tmap_a, bar, m0 + c * 32, x0, oh, img);
                            } else {
                                const int col = n0 + (c - kBM / 32) * 32;
                                const int tap = col / p.ck, ci = col % p.ck;
                                ptx::tma_load_4d(sb + (c - kBM / 32) * 4096u + row_off, &tmap_b, bar, ci,
                                                 x0 + tap % p.taps_s + p.off_w, oh + tap / p.taps_s + p.off_h, img);
                            }
                        }
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
        }
        __syncwarp();
    } else if (warp == 1 || warp == 2) {
        // ------------------------------ MMA issuers ------------------------------
        // One thread can hand the tensor pipe an MMA every ~100-150 cycles, and every barrier wait
        // costs it as much again, so a single issuer with three waits per chunk leaves the pipe idle
        // a third of the time.  Two threads in different warps share the work: warp 1 issues the even
        // chunks (accumulator 0), warp 2 the odd ones (accumulator 1).  A chunk's MMAs depend on no
        // other chunk's, so the two streams need no ordering between them; each thread walks the
        // whole stage ring and acts on its own chunks only.
        //
        // A parity wait tells "phase k is over" from "phase k has not begun" only while the waiter is
        // at most one phase ahead of the barrier.  With three stages and two-stage chunks, the
        // second stage of chunk c+1 is the first stage of chunk c one phase on, so the issuer of
        // chunk c+1 must not look at the stage barriers until the issuer of chunk c has seen that
        // chunk's operands arrive: issue_progress carries that fact from one thread to the other.
        if (lane == 0) {
            const uint32_t who = (uint32_t)(warp - 1);
            const uint32_t idesc = make_idesc(p.a_mn_major, p.b_mn_major);
            // per-MMA advance of the descriptor start address, in 16-byte units
            const uint32_t a_step16 = (p.a_mn_major ? 1024u : (uint32_t)kMmaK * 4u) >> 4;
            const uint32_t b_step16 = (p.b_mn_major ? 1024u : (uint32_t)kMmaK * 4u) >> 4;
            const uint32_t a_lbo = p.a_mn_major ? 4096u : 16u, a_sbo = p.a_mn_major ? 512u : 1024u;
            const uint32_t b_lbo = p.b_mn_major ? 4096u : 16u, b_sbo = p.b_mn_major ? 512u : 1024u;
            const uint32_t a_lay = p.a_mn_major ? kLayoutSw128Base32 : kLayoutSw128;
            const uint32_t b_lay = p.b_mn_major ? kLayoutSw128Base32 : kLayoutSw128;
            const uint32_t a_hi = desc_hi(a_sbo, a_lay), b_hi = desc_hi(b_sbo, b_lay);
            const uint32_t a_lo0 = desc_lo(tiles, a_lbo), b_lo0 = desc_lo(tiles + kABytes, b_lbo);
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_iter = 0;  // chunks issued so far: buffer = acc_iter & 1, phase = (acc_iter >> 1) & 1
            bool dead = false;
            for (int t = blockIdx.x; t < num_work && !dead; t += gridDim.x) {
                const int num_kb = decode_work(p, t).num_kb;
                for (int kb0 = 0; kb0 < num_kb && !dead; kb0 += kChunkKB, ++acc_iter) {
                    const uint32_t acc = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
                    if (acc != who) {  // the other issuer's chunk: step over its stages
                        stage += kb0 + kChunkKB < num_kb ? kChunkKB : num_kb - kb0;
                        if (stage >= kStages) { stage -= kStages; phase ^= 1u; }
                        continue;
                    }
                    if (!ptx::mbar_wait_bounded(acc_empty_bar(acc), acc_phase ^ 1u, kWaitLimit)) {
                        raise_timeout(p, abort_flag);
                        dead = true;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    {   // wait (bounded) until the other issuer is past the stage waits of chunk acc_iter - 1
                        const long long t_begin = clock64();
                        while (issue_progress[who ^ 1u] < acc_iter) {
                            if (clock64() - t_begin > (long long)kWaitLimit) { dead = true; break; }
                        }
                        if (dead) {
                            raise_timeout(p, abort_flag);
                            break;
                        }
                    }
                    const uint32_t d_tmem = tmem_base + acc * kAccCols;
                    const int kb1 = kb0 + kChunkKB < num_kb ? kb0 + kChunkKB : num_kb;
                    for (int kb = kb0; kb < kb1; ++kb) {
                        if (!ptx::mbar_wait_bounded(full_bar(stage), phase, kWaitLimit)) {
                            raise_timeout(p, abort_flag);
                            dead = true;
                            break;
                        }
                        if (kb + 1 == kb1) {  // all of this chunk's operands have arrived
                            __threadfence_block();
                            issue_progress[who] = acc_iter + 1u;
                        }
                        ptx::tc_fence_after_sync();
                        const uint32_t off = (uint32_t)stage * (kStageBytes >> 4);
#pragma unroll
                        for (int k = 0; k < kBK / kMmaK; ++k)
                            ptx::mma_tf32(d_tmem, desc_join(a_hi, a_lo0 + off + k * a_step16), desc_join(b_hi, b_lo0 + off + k * b_step16),
                                          idesc, (kb != kb0 || k != 0) ? 1u : 0u);
                        ptx::mma_commit(empty_bar(stage));  // stage reusable once these MMAs have read it
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                    if (dead) break;
                    ptx::mma_commit(acc_full_bar(acc));      // chunk sum complete
                }
            }
        }
        __syncwarp();
    }
    } else {
        ptx::setmaxnreg_inc<208>();
        // ------------------------------ accumulate + epilogue ------------------------------
        const int quad = warp & 3;             // TMEM lanes [32*quad, 32*quad+32) belong to this warp
        const int half = (warp - 4) >> 2;      // columns [128*half, 128*half+128) of the tile
        uint32_t acc_iter = 0;
        bool dead = false;
        for (int t = blockIdx.x; t < num_work && !dead; t += gridDim.x) {
            const WorkItem w = decode_work(p, t);
            const int m0 = w.m0, n0 = w.n0, num_kb = w.num_kb;
            // rows of C this tile may write, and where split results go
            const int m_end = m0 + p.tile_rows < p.M ? m0 + p.tile_rows : p.M;
            // a piece for the CTA's slot addresses it as if the slot were the tile's place in C
            float* const c_base = w.partial ? p.sk_partials + ((long long)blockIdx.x * p.tile_rows - m0) * p.ldc
                                            : p.C + (long long)w.split * p.split_stride;
            // In mode 1 the C tensor map is [complete tiles][tile_rows][N]; an incomplete last tile
            // takes the scalar path.
            const bool use_tma = p.tma_store && (p.mode != 1 || w.tile_m < p.full_tiles_m);
            // level-1 running sums, two per 64-bit register (packed adds); 0 + x is exact, so a group's
            // first chunk needs no special case
            unsigned long long sum2[64];
#pragma unroll
            for (int j = 0; j < 64; ++j) sum2[j] = 0ull;
            const uint32_t my_stage_addr = out_stage + (uint32_t)(warp - 4) * kOutWarpBytes;
            float* my_stage = reinterpret_cast<float*>(smem_raw + (my_stage_addr - raw));
            const int row0 = m0 + quad * 32;
            int in_group = 0;
            bool flushed = false;
            for (int kb0 = 0; kb0 < num_kb; kb0 += kChunkKB) {
                const uint32_t acc = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
                bool ok = true;
                if (lane == 0) ok = ptx::mbar_wait_bounded(acc_full_bar(acc), acc_phase, kWaitLimit);
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                if (!ok) {
                    if (lane == 0) raise_timeout(p, abort_flag);
                    dead = true;
                    break;
                }
                if (*abort_flag) { dead = true; break; }
                ptx::tc_fence_after_sync();
                const uint32_t tbase = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * kAccCols + (uint32_t)half * 128u;
                // Two 32-column loads in flight per wait; the TMEM buffer is handed back to the MMA
                // warp as soon as its last values are in registers, before they are added.
#pragma unroll
                for (int pair = 0; pair < 2; ++pair) {
                    uint32_t ra[32], rb[32];
                    ptx::tmem_load_32cols(tbase + pair * 64, ra);
                    ptx::tmem_load_32cols(tbase + pair * 64 + 32, rb);
                    ptx::tmem_load_wait();
                    if (pair == 1) {
                        ptx::tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(acc_empty_bar(acc));
                    }
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        ptx::add2_rn(sum2[pair * 32 + j / 2], ra[j], ra[j + 1]);
                        ptx::add2_rn(sum2[pair * 32 + 16 + j / 2], rb[j], rb[j + 1]);
                    }
                }
                ++acc_iter;
                const bool last = kb0 + kChunkKB >= num_kb;
                if (!last && ++in_group < kFlushChunks) continue;
                // ---- move the level-1 sums to C (level 2): registers -> swizzled shared boxes -> TMA.
                // The first group of a tile is stored, later groups are added at the destination.
                if (kEpi)
                    epi_transform(sum2, p, row0 + lane < m_end, n0 + half * 128, reinterpret_cast<uint32_t*>(my_stage), epi_hist, lane);
                if (use_tma && flushed) {
                    if (lane == 0) ptx::bulk_wait_all();  // the earlier store/add to these addresses is complete
                }
#pragma unroll
                for (int pass = 0; pass < 4; ++pass) {
                    const int col0 = n0 + half * 128 + pass * kOutCols;
                    float* box = my_stage + (pass & 1) * 1024;
                    // at most the newest copy (it reads the other box) may still be reading
                    if (lane == 0) ptx::bulk_wait_read_1();
                    __syncwarp();
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const int j = pass * kOutCols + c * 4;
                        const float2 v0 = ptx::unpack2(sum2[j / 2]), v1 = ptx::unpack2(sum2[j / 2 + 1]);
                        *reinterpret_cast<float4*>(box + lane * 32 + ((c ^ (lane & 7)) << 2)) =
                            make_float4(v0.x, v0.y, v1.x, v1.y);
                    }
                    if (use_tma) {
                        ptx::fence_proxy_async();
                        __syncwarp();
                        if (lane == 0) {
                            if (row0 < m_end && col0 < p.N) {
                                const uint32_t src = my_stage_addr + (pass & 1) * kOutBoxBytes;
                                const int y = p.mode == 1 ? quad * 32 : row0;
                                const int z = w.partial ? (int)blockIdx.x : (p.mode == 1 ? w.tile_m : w.split);
                                const CUtensorMap* cm = w.partial ? &tmap_p : &tmap_c;
                                if (flushed) ptx::tma_reduce_add_3d(cm, src, col0, y, z);
                                else ptx::tma_store_3d(cm, src, col0, y, z);
                            }
                            ptx::bulk_commit();  // committed even when empty: the wait above counts groups
                        }
                    } else {
                        __syncwarp();
                        for (int r = 0; r < 32; ++r) {
                            const int row = row0 + r;
                            if (row >= m_end) break;
                            const int c = lane;
                            if (col0 + c < p.N) {
                                float* g = c_base + (long long)row * p.ldc + col0 + c;
                                const float v = box[r * 32 + (((c >> 2) ^ (r & 7)) << 2) + (c & 3)];
                                *g = flushed ? __fadd_rn(*g, v) : v;
                            }
                        }
                        __syncwarp();
                    }
                }
                flushed = true;
                in_group = 0;
                if (!last) {
#pragma unroll
                    for (int j = 0; j < 64; ++j) sum2[j] = 0ull;
                }
            }
            if (dead) break;
        }
        if (lane == 0) ptx::bulk_wait_read_all();  // shared memory stays valid until the last copy has read it
        __syncwarp();
    }

    // ------------------------------ common exit ------------------------------
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (kEpi) epi_merge(p, epi_hist);
    if (*abort_flag) {
        // give TMA copies that may still be in flight time to land before the CTA's shared
        // memory is handed to another CTA
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// CTA-pair variant (dense products): two CTAs of a cluster share one 256 x 256 tile.
//
// Each CTA stages its own 128 rows of op(A) and its own 128 columns of op(B) (32 KB per stage
// instead of 48), the leader CTA's two MMA threads issue tcgen05.mma.cta_group::2 with M = 256,
// and each CTA's tensor memory receives its 128 x 256 half of the accumulator.  Per MMA a CTA
// feeds 8 KB of operands from shared memory instead of 12 KB.  Nothing is copied between the
// CTAs; they only signal each other's barriers:
//   full[s]      (leader's) two arrivals, one per CTA's producer with that CTA's byte count;
//                both CTAs' TMA loads credit their bytes to it
//   empty[s]     (each CTA's own) one arrival from the MMA commit, sent to both CTAs
//   acc_full[b]  (each CTA's own) one arrival from the MMA commit, sent to both CTAs
//   acc_empty[b] (leader's) sixteen arrivals: the eight accumulate warps of both CTAs
// The three-level summation and the output path are those of the single-CTA kernel.
// ------------------------------------------------------------------------------------------------
#ifndef QFMT_PSTAGES
#define QFMT_PSTAGES 5
#endif
#ifndef QFMT_POUT_BLOCKS
#define QFMT_POUT_BLOCKS 2
#endif
constexpr int kPStages = QFMT_PSTAGES;
constexpr uint32_t kPABytes = kBM * kBK * 4;          // 128 rows of A
constexpr uint32_t kPBBytes = (kBN / 2) * kBK * 4;    // 128 of the tile's 256 columns of B
constexpr uint32_t kPStageBytes = kPABytes + kPBBytes;
// Output staging of the pair kernel.  When N is a multiple of 32, C is described to the copy engine as
// {32 columns, rows, N / 32 column blocks, splits}, and one copy moves kPOutBlocks 32 x 32 blocks of a
// warp's 32 x 128 patch: with kPOutBlocks = 4 the whole patch is staged at once (16 KB per warp) and a
// flush costs the copy engine eight instructions per CTA instead of thirty-two.
constexpr int kPOutBlocks = QFMT_POUT_BLOCKS;
constexpr uint32_t kPOutWarpBytes = (kPOutBlocks * kOutBoxBytes > kOutWarpBytes) ? kPOutBlocks * kOutBoxBytes : kOutWarpBytes;
constexpr uint32_t kPOutBytes = kAccWarps * kPOutWarpBytes;
// Balanced schedule: a pair's pieces (at most kMaxSkPieces) are worked out once, by the first threads of
// each CTA, into a table in shared memory that every role then reads.
constexpr int kMaxSkPieces = 64;
constexpr uint32_t kSkTableBytes = kMaxSkPieces * 16;
constexpr uint32_t kPairSmemBytes = kPStages * kPStageBytes + kPOutBytes + 1024 + 256 + kEpiHistBytes + kSkTableBytes;
static_assert(kPairSmemBytes <= 232448, "pair kernel: shared memory");
// The two MMA issuers of the pair kernel tell a stage's phases apart without a progress word only
// when the ring has at least four stages (see the issuer's comment); three stages gave wrong sums.
static_assert(kPStages >= 4, "pair kernel: at least four stages");
static_assert(4 % kPOutBlocks == 0, "pair kernel: a warp's four column blocks in whole copies");

// Operand kinds of the pair kernel: fp32 containers read as TF32, or packed 16-bit codes that are
// binary16 (1/5/10) or bfloat16 (1/8/7) words.  A stage is one 128-byte swizzle row per operand row
// in every kind: 32 TF32 or 64 16-bit K elements, four MMAs.
enum : int { kKindTf32 = 0, kKindF16 = 1, kKindBf16 = 2 };
__device__ __forceinline__ uint32_t make_idesc_pair(int a_mn, int b_mn, int kind) {
    const uint32_t ab = kind == kKindTf32 ? 2u : (kind == kKindF16 ? 0u : 1u);  // A, B format field
    return (1u << 4) | (ab << 7) | (ab << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16)
           | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)((2 * kBM) >> 4) << 24);
}

// kMode 0: dense operands.  kMode 1: forward / data gradient of a convolution (see conv_device): each
// CTA of the pair owns one M-tile of whole image rows (p.rows_per_blk rows, p.conv_rows pixels) and
// half of the 256 filter columns; its pixel operand arrives as one box per image touched from
// row_maps, C is written through tmap_c ({32, conv_rows, N / 32, complete tiles}: rows past the tile
// are clipped) or, for the incomplete last tile, tmap_c2.  kMode 2: filter gradient of a convolution with
// padded stages (GemmParams::wg_padded): a dense product of two MN-major operands whose stages are
// gathered pixel rows, C_out is M (128 rows per CTA), (tap, C_in) is N (128 columns per CTA, inside one
// tap), one rank-5 copy per operand and stage.
// kSk: the balanced schedule (GemmParams::sk_flags) is compiled in; products that do not use it run an
// instantiation without any of its code.
template <bool kEpi, int kKind, int kMode, bool kSk>
__device__ __forceinline__ void pair_body(const CUtensorMap& tmap_a, const CUtensorMap& tmap_b, const CUtensorMap& tmap_c,
                                          const CUtensorMap* tmap_c2, const CUtensorMap* row_maps, const GemmParams& p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = ptx::smem_addr(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    const uint32_t out_stage = tiles + kPStages * kPStageBytes;
    const uint32_t bars = out_stage + kPOutBytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kPStages + s); };
    auto acc_full_bar = [&](int a) { return bars + 8u * (2 * kPStages + a); };
    auto acc_empty_bar = [&](int a) { return bars + 8u * (2 * kPStages + 2 + a); };
    // balanced schedule: head_bar (the non-leader CTA's) collects the pair's accumulate warps whose stores
    // of a tile's first piece are complete, tail_bar tells a CTA's accumulate warps that the pair before
    // has stored the first piece of their tile
    const uint32_t head_bar = bars + 8u * (2 * kPStages + 4), tail_bar = bars + 8u * (2 * kPStages + 5);
    uint8_t* gen_bars = smem_raw + (bars - raw);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen_bars + 8 * (2 * kPStages + 6));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen_bars + 8 * (2 * kPStages + 6) + 8);
    uint32_t* epi_hist = reinterpret_cast<uint32_t*>(gen_bars + 256);
    int4* const sk_table = reinterpret_cast<int4*>(gen_bars + 256 + kEpiHistBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t rank = ptx::cluster_ctarank();  // 0 = leader
    if (kEpi) {
        for (int i = threadIdx.x; i < kEpiBins; i += kThreads) epi_hist[i] = 0u;
    }
    const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
    if (kSk) {
        // piece j of this pair: {tile, first stage, stages, partial | head << 1}
        if ((int)threadIdx.x < p.sk_pieces) {
            const PairPiece pc = pair_piece(p.sk_q, p.sk_r, p.sk_cpt, p.kb_total, num_clusters, cluster_id, (int)threadIdx.x);
            sk_table[threadIdx.x] = make_int4(pc.tile, pc.kb_begin, pc.num_kb, pc.partial | (pc.head << 1));
        }
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPStages; ++s) {
            ptx::mbar_init(full_bar(s), 2);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(acc_full_bar(a), 1);
            ptx::mbar_init(acc_empty_bar(a), 2 * kAccWarps);
        }
        ptx::mbar_init(head_bar, 2 * kAccWarps);  // used in the non-leader CTA: the accumulate warps of both
        ptx::mbar_init(tail_bar, 1);
        *abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_a);
        ptx::prefetch_tensormap(&tmap_b);
        if (p.tma_store) ptx::prefetch_tensormap(&tmap_c);
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
        ptx::tmem_relinquish_pair();
    }
    // Everything above touched shared and tensor memory only and may run while the kernel before this one
    // in the stream drains; from here on global memory is read and written.
    grid_dependency_wait();
    announce_launch(p.status, p.launch_tag);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();  // the peer's barriers exist before anything is signalled to them
    ptx::tc_fence_after_sync();
    grid_launch_dependents();
    const uint32_t tmem_base = *tmem_slot;
    // work items of this pair: its pieces under the balanced schedule (t = 0, 1, ...), else every
    // num_clusters-th tile (t = cluster_id, cluster_id + num_clusters, ...)
    const int t_begin = kSk ? 0 : cluster_id, t_step = kSk ? 1 : num_clusters;
    const int t_end = kSk ? p.sk_pieces : p.tiles_m * p.tiles_n * p.splits;
    auto work_item = [&](int j) -> WorkItem {
        if (kSk) {
            const int4 e = sk_table[j];
            WorkItem w;
            w.split = 0;
            w.tile_m = e.x % p.tiles_m;
            w.tile_n = e.x / p.tiles_m;
            w.m0 = w.tile_m * p.tile_rows;
            w.n0 = w.tile_n * kBN;
            w.kb_begin = e.y;
            w.num_kb = e.z;
            w.partial = e.w & 1;
            w.head = e.w >> 1;
            return w;
        }
        return decode_work(p, j);
    };

    if (warp < 4) {
    ptx::setmaxnreg_dec<56>();
    if (warp == 0 || warp == 3) {
        // ------------------------------ TMA producers (both CTAs) ------------------------------
        // One thread needs ~700 cycles for a dense stage (the wait on its slot, the byte count, two
        // copies) and over 1000 for a convolution's (tap arithmetic, a copy per image touched), and the
        // tensor pipe consumes a stage in 512, so two threads fill alternate stages: warp 0 the even
        // ones of the CTA's stage sequence, warp 3 the odd ones.
        if (lane == 0) {
            const uint32_t who = warp == 0 ? 0u : 1u;
            uint32_t seq = 0;
            int stage = 0;
            uint32_t phase = 0;
            for (int t = t_begin; t < t_end && !*abort_flag; t += t_step) {
                const WorkItem w = work_item(t);
                const int m0 = w.m0 + (int)rank * kBM, n0 = w.n0 + (int)rank * (kBN / 2);
                // convolution: the boxes of this CTA's M-tile (one per image it touches: first row within
                // the image, image, rows) and the tap / channel block of the piece's first stage; the
                // stage loop then only counts
                int box_h[3], box_img[3], box_cnt[3], n_boxes = 0;
                int tap = 0, cb = 0, tap_r = 0, tap_s = 0;
                if (kMode == 1) {
                    const int ctile = 2 * w.tile_m + (int)rank;
                    int j = 0;
                    while (j < p.rows_per_blk && n_boxes < 3) {
                        const int q = ctile * p.rows_per_blk + j;
                        const int h = q % p.img_rows;
                        int cnt = p.rows_per_blk - j;
                        if (cnt > p.img_rows - h) cnt = p.img_rows - h;
                        if (cnt > kMaxRowMaps) cnt = kMaxRowMaps;
                        box_h[n_boxes] = h; box_img[n_boxes] = q / p.img_rows; box_cnt[n_boxes] = cnt;
                        ++n_boxes;
                        j += cnt;
                    }
                    if (j < p.rows_per_blk) n_boxes = -1;  // more than three boxes: worked out per stage below
                    tap = w.kb_begin / p.cblocks; cb = w.kb_begin % p.cblocks;
                    tap_r = tap / p.taps_s; tap_s = tap % p.taps_s;
                }
                for (int kb = w.kb_begin; kb < w.kb_begin + w.num_kb; ++kb) {
                    const int my_tap = tap, my_cb = cb, my_r = tap_r, my_s = tap_s;
                    if (kMode == 1) {  // the next stage's tap and channel block
                        if (++cb == p.cblocks) {
                            cb = 0; ++tap;
                            if (++tap_s == p.taps_s) { tap_s = 0; ++tap_r; }
                        }
                    }
                    if ((seq++ & 1u) != who) {  // the other producer's stage
                        if (++stage == kPStages) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    if (!ptx::mbar_wait_bounded(empty_bar(stage), phase ^ 1u, kWaitLimit)) {
                        raise_timeout(p, abort_flag);
                        break;
                    }
                    const uint32_t sa = tiles + stage * kPStageBytes;
                    const uint32_t sb = sa + kPABytes;
                    const uint32_t bar = ptx::map_to_cta(full_bar(stage), 0);  // the leader's barrier
                    const int k0 = kb * (kKind == kKindTf32 ? kBK : 2 * kBK);
                    if (kMode == 1) {
                        ptx::mbar_expect_tx_cluster(bar, p.a_bytes + kPBBytes);
                        // A: this CTA's image rows at the tap's offset, one box per image touched (rows and
                        // columns outside the image, and images past the batch, read as zero)
                        const int dh = p.tap_sign * my_r + p.off_h, dw = p.tap_sign * my_s + p.off_w;
                        uint32_t dst = sa;
#pragma unroll
                        for (int b = 0; b < 3; ++b) {
                            if (b < n_boxes) {
                                ptx::tma_load_4d_pair(dst, &row_maps[box_cnt[b] - 1], bar, my_cb * 32, dw, box_h[b] + dh, box_img[b]);
                                dst += (uint32_t)(box_cnt[b] * p.img_w) * 128u;
                            }
                        }
                        if (n_boxes < 0) {
                            const int ctile = 2 * w.tile_m + (int)rank;
                            int j = 0;
                            while (j < p.rows_per_blk) {
                                const int q = ctile * p.rows_per_blk + j;
                                const int h = q % p.img_rows, img = q / p.img_rows;
                                int cnt = p.rows_per_blk - j;
                                if (cnt > p.img_rows - h) cnt = p.img_rows - h;
                                if (cnt > kMaxRowMaps) cnt = kMaxRowMaps;
                                ptx::tma_load_4d_pair(sa + (uint32_t)(j * p.img_w) * 128u, &row_maps[cnt - 1], bar, my_cb * 32, dw,
                                                      h + dh, img);
                                j += cnt;
                            }
                        }
                        if (p.b_mn_major) ptx::tma_load_4d_pair(sb, &tmap_b, bar, 0, my_tap, my_cb * 32, n0 >> 5);
                        else ptx::tma_load_2d_pair(sb, &tmap_b, bar, my_tap * p.ck + my_cb * 32, n0);
                        if (++stage == kPStages) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    ptx::mbar_expect_tx_cluster(bar, kPStageBytes);
                    if (kMode == 2) {
                        // stage kb = rows_per_blk output rows of one image, each padded to a power-of-two number of
                        // K rows; A = output gradient, B = activations at the tap this CTA's columns belong to
                        const int q = kb * p.rows_per_blk;
                        const int oh = q % p.img_rows, img = q / p.img_rows;
                        const int tap = n0 / p.ck, ci = n0 % p.ck;
                        ptx::tma_load_5d_pair(sa, &tmap_a, bar, 0, 0, oh, img, m0 >> 5);
                        ptx::tma_load_5d_pair(sb, &tmap_b, bar, 0, tap % p.taps_s + p.off_w, oh + tap / p.taps_s + p.off_h, img,
                                              ci >> 5);
                        if (++stage == kPStages) { stage = 0; phase ^= 1u; }
                        continue;
                    }
                    // an MN-major operand arrives as column blocks of one 128-byte row per K element:
                    // 32 columns x 32 K rows (TF32) or 64 columns x 64 K rows (16-bit codes)
                    constexpr int kBlkShift = kKind == kKindTf32 ? 5 : 6, kBlk = 1 << kBlkShift;
                    constexpr uint32_t kBlkBytes = kKind == kKindTf32 ? 4096u : 8192u;
                    if (p.a_blocked) {
                        ptx::tma_load_3d_pair(sa, &tmap_a, bar, 0, k0, m0 >> kBlkShift);
                    } else if (p.a_mn_major) {
                        for (int c = 0; c < kBM / kBlk; ++c)
                            ptx::tma_load_2d_pair(sa + c * kBlkBytes, &tmap_a, bar, m0 + c * kBlk, k0);
                    } else {
                        ptx::tma_load_2d_pair(sa, &tmap_a, bar, k0, m0);
                    }
                    if (p.b_blocked) {
                        ptx::tma_load_3d_pair(sb, &tmap_b, bar, 0, k0, n0 >> kBlkShift);
                    } else if (p.b_mn_major) {
                        for (int c = 0; c < (kBN / 2) / kBlk; ++c)
                            ptx::tma_load_2d_pair(sb + c * kBlkBytes, &tmap_b, bar, n0 + c * kBlk, k0);
                    } else {
                        ptx::tma_load_2d_pair(sb, &tmap_b, bar, k0, n0);
                    }
                    if (++stage == kPStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1 || warp == 2) {
        // ------------------------------ MMA issuers (leader CTA only) ------------------------------
        // Two issuers on alternating chunks, as in the single-CTA kernel.  No progress word is needed
        // here: an issuer reaches chunk c+1 only after the accumulate warps have drained chunk c-1,
        // hence after chunk c-2 was issued in full, and with a ring of five stages the previous
        // phase of the stages of chunk c+1 belongs to chunks c-2 and c-1.
        if (kSk && lane == 0 && rank == 1 && warp == 1) {
            // ---- balanced schedule: hand-over between pairs (this warp has no MMAs to issue in the
            // non-leader CTA).  A tile cut by a range boundary is begun by one pair (its first piece,
            // "head") and finished by the next (its last piece, which adds at the destination).
            // Once the sixteen accumulate warps of this pair have completed their stores of a head
            // piece this thread raises the next pair's flag; before this pair's accumulate warps may
            // add a piece that begins inside a tile it waits for this pair's own flag and then lets
            // both CTAs go on.
            bool dead = false;
            for (int t = t_begin; t < t_end && !dead; t += t_step) {
                const WorkItem w = work_item(t);
                if (w.num_kb <= 0) continue;
                if (w.head) {
                    if (!ptx::mbar_wait_bounded(head_bar, 0u, kWaitLimit)) {
                        raise_timeout(p, abort_flag);
                        break;
                    }
                    ptx::fence_proxy_async_all();
                    __threadfence();
                    *reinterpret_cast<volatile int*>(p.sk_flags + (cluster_id + 1) * 16) = 1;
                }
                if (w.partial) {
                    volatile int* flag = p.sk_flags + cluster_id * 16;
                    const long long t_begin_wait = clock64();
                    while (*flag == 0 && !*abort_flag) {
                        if (clock64() - t_begin_wait > (long long)kWaitLimit) { dead = true; break; }
                        __nanosleep(64);
                    }
                    if (dead) {
                        raise_timeout(p, abort_flag);
                        break;
                    }
                    __threadfence();
                    ptx::mbar_arrive(tail_bar);
                    ptx::mbar_arrive_cluster(ptx::map_to_cta(tail_bar, 0));
                }
            }
        }
        if (lane == 0 && rank == 0) {
            const uint32_t who = (uint32_t)(warp - 1);
            const uint32_t idesc = make_idesc_pair(p.a_mn_major, p.b_mn_major, kKind);
            // per-MMA advance of the descriptor start address, in 16-byte units
            // MN-major operand: the leading offset is the pitch of its column blocks, the stride offset
            // that of eight K rows, and one MMA consumes 8 (TF32) or 16 (16-bit) K rows of 128 bytes.
            // TF32 needs the 32-byte-atom form of the 128-byte swizzle there, 16-bit codes the plain one.
            constexpr bool k16 = kKind != kKindTf32;
            constexpr uint32_t mn_step = k16 ? 2048u : 1024u, mn_lbo = k16 ? 8192u : 4096u, mn_sbo = k16 ? 1024u : 512u;
            constexpr uint32_t mn_lay = k16 ? kLayoutSw128 : kLayoutSw128Base32;
            const uint32_t a_step16 = (p.a_mn_major ? mn_step : (uint32_t)kMmaK * 4u) >> 4;
            const uint32_t b_step16 = (p.b_mn_major ? mn_step : (uint32_t)kMmaK * 4u) >> 4;
            const uint32_t a_lbo = p.a_mn_major ? mn_lbo : 16u, a_sbo = p.a_mn_major ? mn_sbo : 1024u;
            const uint32_t b_lbo = p.b_mn_major ? mn_lbo : 16u, b_sbo = p.b_mn_major ? mn_sbo : 1024u;
            const uint32_t a_lay = p.a_mn_major ? mn_lay : kLayoutSw128;
            const uint32_t b_lay = p.b_mn_major ? mn_lay : kLayoutSw128;
            const uint32_t a_hi = desc_hi(a_sbo, a_lay), b_hi = desc_hi(b_sbo, b_lay);
            const uint32_t a_lo0 = desc_lo(tiles, a_lbo), b_lo0 = desc_lo(tiles + kPABytes, b_lbo);
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_iter = 0;
            bool dead = false;
            for (int t = t_begin; t < t_end && !dead; t += t_step) {
                const int num_kb = kSk ? sk_table[t].z : decode_work(p, t).num_kb;
                for (int kb0 = 0; kb0 < num_kb && !dead; kb0 += kChunkKB, ++acc_iter) {
                    const uint32_t acc = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
                    if (acc != who) {  // the other issuer's chunk: step over its stages
                        stage += kb0 + kChunkKB < num_kb ? kChunkKB : num_kb - kb0;
                        if (stage >= kPStages) { stage -= kPStages; phase ^= 1u; }
                        continue;
                    }
                    if (!ptx::mbar_wait_bounded(acc_empty_bar(acc), acc_phase ^ 1u, kWaitLimit)) {
                        raise_timeout(p, abort_flag);
                        dead = true;
                        break;
                    }
                    ptx::tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + acc * kAccCols;
                    const int kb1 = kb0 + kChunkKB < num_kb ? kb0 + kChunkKB : num_kb;
                    for (int kb = kb0; kb < kb1; ++kb) {
                        if (!ptx::mbar_wait_bounded(full_bar(stage), phase, kWaitLimit)) {
                            raise_timeout(p, abort_flag);
                            dead = true;
                            break;
                        }
                        ptx::tc_fence_after_sync();
                        const uint32_t off = (uint32_t)stage * (kPStageBytes >> 4);
#pragma unroll
                        for (int k = 0; k < kBK / kMmaK; ++k) {
                            const uint64_t da = desc_join(a_hi, a_lo0 + off + k * a_step16);
                            const uint64_t db = desc_join(b_hi, b_lo0 + off + k * b_step16);
                            if (kKind == kKindTf32) ptx::mma_tf32_pair(d_tmem, da, db, idesc, (kb != kb0 || k != 0) ? 1u : 0u);
                            else ptx::mma_f16_pair(d_tmem, da, db, idesc, (kb != kb0 || k != 0) ? 1u : 0u);
                        }
                        ptx::mma_commit_pair(empty_bar(stage), 3);  // both CTAs may refill this stage
                        if (++stage == kPStages) { stage = 0; phase ^= 1u; }
                    }
                    if (dead) break;
                    ptx::mma_commit_pair(acc_full_bar(acc), 3);      // chunk sum complete in both CTAs
                }
            }
        }
        __syncwarp();
    }
    } else {
        // 128 x 56 + 256 x 224 registers are exactly the 384 x 168 the CTA was launched with; the increase
        // blocks until that many are free in the CTA's own pool, so a larger request would never return.
        // The accumulate warps hold 128 sums and 64 freshly loaded values; with 208 registers a few
        // more live values in their loop already spilled (measured: 12 % slower products).
        ptx::setmaxnreg_inc<224>();
        // ------------------------------ accumulate + epilogue (both CTAs) ------------------------------
        const int quad = warp & 3;
        const int half = (warp - 4) >> 2;
        const uint32_t my_stage_addr = out_stage + (uint32_t)(warp - 4) * kPOutWarpBytes;
        float* const my_stage = reinterpret_cast<float*>(smem_raw + (my_stage_addr - raw));
        uint32_t acc_iter = 0;
        bool dead = false;
        for (int t = t_begin; t < t_end && !dead; t += t_step) {
            const WorkItem w = work_item(t);
            constexpr bool kConv = kMode == 1;
            const int cta_rows = kConv ? p.conv_rows : kBM;  // rows of C this CTA owns in the tile
            const int m0 = w.m0 + (int)rank * cta_rows, n0 = w.n0;
            const int m_end = m0 + cta_rows < p.M ? m0 + cta_rows : p.M;
            float* const c_base = p.C + (long long)w.split * p.split_stride;
            const bool use_tma = p.tma_store != 0;
            const int row0 = m0 + quad * 32;
            // a piece that begins inside its tile adds to what the pair before has stored there
            bool flushed = kSk && w.partial != 0;
            // The piece's chunks in groups of kFlushChunks: a group's chunk sums are added up in registers
            // (the inner loop holds nothing else), then the group moves to C.
            const int chunks = (w.num_kb + kChunkKB - 1) / kChunkKB;
            for (int c0 = 0; c0 < chunks; c0 += kFlushChunks) {
                // level-1 running sums, two per 64-bit register (packed adds); 0 + x is exact, so a group's
                // first chunk needs no special case
                unsigned long long sum2[64];
#pragma unroll
                for (int j = 0; j < 64; ++j) sum2[j] = 0ull;
                const int c1 = c0 + kFlushChunks < chunks ? c0 + kFlushChunks : chunks;
                for (int c = c0; c < c1; ++c) {
                    const uint32_t acc = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
                    bool ok = true;
                    if (lane == 0) ok = ptx::mbar_wait_bounded(acc_full_bar(acc), acc_phase, kWaitLimit);
                    ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                    if (!ok) {
                        if (lane == 0) raise_timeout(p, abort_flag);
                        dead = true;
                        break;
                    }
                    if (*abort_flag) { dead = true; break; }
                    ptx::tc_fence_after_sync();
                    const uint32_t tbase = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * kAccCols + (uint32_t)half * 128u;
#pragma unroll
                    for (int pair = 0; pair < 2; ++pair) {
                        uint32_t ra[32], rb[32];
                        ptx::tmem_load_32cols(tbase + pair * 64, ra);
                        ptx::tmem_load_32cols(tbase + pair * 64 + 32, rb);
                        ptx::tmem_load_wait();
                        if (pair == 1) {
                            ptx::tc_fence_before_sync();
                            __syncwarp();
                            if (lane == 0) ptx::mbar_arrive_cluster(ptx::map_to_cta(acc_empty_bar(acc), 0));
                        }
#pragma unroll
                        for (int j = 0; j < 32; j += 2) {
                            ptx::add2_rn(sum2[pair * 32 + j / 2], ra[j], ra[j + 1]);
                            ptx::add2_rn(sum2[pair * 32 + 16 + j / 2], rb[j], rb[j + 1]);
                        }
                    }
                    ++acc_iter;
                }
                if (dead) break;
                // ---- the group's sums move to C: registers -> swizzled staging -> TMA (stored for the
                // first group of a tile, added at the destination for later ones)
                if (kEpi)
                    epi_transform(sum2, p, row0 + lane < m_end, n0 + half * 128, reinterpret_cast<uint32_t*>(my_stage), epi_hist, lane);
                if (kSk && w.partial && c0 == 0) {
                    // the pair before this one has stored the first piece of this tile (warp 3 watches its flag)
                    bool seen = true;
                    if (lane == 0) seen = ptx::mbar_wait_bounded(tail_bar, 0u, kWaitLimit);
                    seen = __shfl_sync(0xFFFFFFFFu, seen ? 1 : 0, 0) != 0;
                    if (!seen) {
                        if (lane == 0) raise_timeout(p, abort_flag);
                        dead = true;
                        break;
                    }
                }
                if (use_tma && flushed) {
                    if (lane == 0) ptx::bulk_wait_all();  // the earlier store/add to these addresses is complete
                }
                if (p.c_blocked) {
                    // Whole copies of kPOutBlocks column blocks: the staging area is filled (each 32 x 32 block
                    // in the swizzled layout of a one-block box), then ONE copy instruction stores it or adds
                    // it at the destination.  Blocks past N and rows past M are clipped by the copy engine.
#pragma unroll
                    for (int pass = 0; pass < 4 / kPOutBlocks; ++pass) {
                        if (lane == 0) ptx::bulk_wait_read_all();  // the previous copy has read the staging area
                        __syncwarp();
#pragma unroll
                        for (int blk = 0; blk < kPOutBlocks; ++blk) {
                            float* box = my_stage + blk * 1024;
#pragma unroll
                            for (int cc = 0; cc < 8; ++cc) {
                                const int j = (pass * kPOutBlocks + blk) * kOutCols + cc * 4;
                                const float2 v0 = ptx::unpack2(sum2[j / 2]), v1 = ptx::unpack2(sum2[j / 2 + 1]);
                                *reinterpret_cast<float4*>(box + lane * 32 + ((cc ^ (lane & 7)) << 2)) =
                                    make_float4(v0.x, v0.y, v1.x, v1.y);
                            }
                        }
                        ptx::fence_proxy_async();
                        __syncwarp();
                        if (lane == 0) {
                            const int cblk = ((n0 + half * 128) >> 5) + pass * kPOutBlocks;
                            if (row0 < m_end && cblk * 32 < p.N) {
                                // convolution: the CTA's own tile of the per-tile map (or the map of the incomplete last tile)
                                const int ctile = 2 * w.tile_m + (int)rank;
                                const bool whole = !kConv || ctile < p.full_tiles_m;
                                const CUtensorMap* cm = whole ? &tmap_c : tmap_c2;
                                const int ry = kConv ? quad * 32 : row0, rz = kConv ? (whole ? ctile : 0) : w.split;
                                if (flushed) ptx::tma_reduce_add_4d(cm, my_stage_addr, 0, ry, cblk, rz);
                                else ptx::tma_store_4d(cm, my_stage_addr, 0, ry, cblk, rz);
                            }
                            ptx::bulk_commit();  // committed even when empty: the waits count groups
                        }
                    }
                } else {
#pragma unroll
                    for (int pass = 0; pass < 4; ++pass) {
                        const int col0 = n0 + half * 128 + pass * kOutCols;
                        float* box = my_stage + (pass & 1) * 1024;
                        if (lane == 0) ptx::bulk_wait_read_1();  // at most the newest copy (it reads the other box) may still be reading
                        __syncwarp();
#pragma unroll
                        for (int cc = 0; cc < 8; ++cc) {
                            const int j = pass * kOutCols + cc * 4;
                            const float2 v0 = ptx::unpack2(sum2[j / 2]), v1 = ptx::unpack2(sum2[j / 2 + 1]);
                            *reinterpret_cast<float4*>(box + lane * 32 + ((cc ^ (lane & 7)) << 2)) =
                                make_float4(v0.x, v0.y, v1.x, v1.y);
                        }
                        if (use_tma) {
                            ptx::fence_proxy_async();
                            __syncwarp();
                            if (lane == 0) {
                                if (row0 < m_end && col0 < p.N) {
                                    const uint32_t src = my_stage_addr + (pass & 1) * kOutBoxBytes;
                                    if (flushed) ptx::tma_reduce_add_3d(&tmap_c, src, col0, row0, w.split);
                                    else ptx::tma_store_3d(&tmap_c, src, col0, row0, w.split);
                                }
                                ptx::bulk_commit();
                            }
                        } else {
                            __syncwarp();
                            for (int r = 0; r < 32; ++r) {
                                const int row = row0 + r;
                                if (row >= m_end) break;
                                if (col0 + lane < p.N) {
                                    float* g = c_base + (long long)row * p.ldc + col0 + lane;
                                    const float v = box[r * 32 + (((lane >> 2) ^ (r & 7)) << 2) + (lane & 3)];
                                    *g = flushed ? __fadd_rn(*g, v) : v;
                                }
                            }
                            __syncwarp();
                        }
                    }
                }
                flushed = true;
            }
            if (dead) break;
            if (kSk && w.head && chunks > 0) {
                // this warp's part of the tile's first piece is in C (its copies have completed)
                if (lane == 0) {
                    ptx::bulk_wait_all();
                    __threadfence();
                    ptx::mbar_arrive_cluster(ptx::map_to_cta(head_bar, 1));
                }
                __syncwarp();
            }
        }
        // shared memory stays valid until the last copy has read it; the copies' writes are complete when
        // the kernel is
        if (lane == 0) ptx::bulk_wait_read_all();
        __syncwarp();
    }

    // ------------------------------ common exit ------------------------------
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (kEpi) epi_merge(p, epi_hist);
    if (*abort_flag) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    }
    ptx::cluster_sync();  // neither CTA leaves while the other may still signal it
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

template <bool kEpi, int kKind, bool kSk>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tf32_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                      const __grid_constant__ CUtensorMap tmap_c, const GemmParams p) {
    pair_body<kEpi, kKind, 0, kSk>(tmap_a, tmap_b, tmap_c, nullptr, nullptr, p);
}

// Forward / data gradient of a convolution on CTA pairs (its own instantiation, so that the dense
// products carry none of its code).
// Filter gradient of a convolution on CTA pairs (padded stages; its own instantiation).
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_wgrad_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                       const __grid_constant__ CUtensorMap tmap_c, const GemmParams p) {
    pair_body<false, kKindTf32, 2, false>(tmap_a, tmap_b, tmap_c, nullptr, nullptr, p);
}

template <bool kSk>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_conv_pair_kernel(const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ CUtensorMap tmap_c,
                      const __grid_constant__ CUtensorMap tmap_c2, const __grid_constant__ RowMaps row_maps,
                      const GemmParams p) {
    pair_body<false, kKindTf32, 1, kSk>(row_maps.m[0], tmap_b, tmap_c, &tmap_c2, row_maps.m, p);
}

// ---- host side ----------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// fp32 tensor map of rank 2..5 with dim0 contiguous; strides in elements for dims 1..rank-1; zero
// fill out of bounds.  Swizzle: 16-byte chunks within 128 bytes for K-major operand tiles and for
// C, 32-byte chunks for MN-major operand tiles.
int make_map(CUtensorMap* map, const float* base, int rank, const uint64_t* dims, const uint64_t* strides_elems,
             const uint32_t* box, bool mn_major) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) { set_last_cuda_error((int)cudaErrorSymbolNotFound); return QFMT_ERR_CUDA; }
    cuuint64_t d[5], st[4];
    cuuint32_t bx[5], estr[5] = {1, 1, 1, 1, 1};
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; bx[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) st[i] = strides_elems[i] * sizeof(float);
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, const_cast<float*>(base), d, st, bx, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE,
                    mn_major ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_last_cuda_error(100000 + (int)r); return QFMT_ERR_CUDA; }
    return QFMT_OK;
}

int make_map_2d(CUtensorMap* map, const float* base, uint64_t dim0, uint64_t dim1, uint64_t ld_elems,
                uint32_t box0, uint32_t box1, bool mn_major) {
    const uint64_t dims[2] = {dim0, dim1}, strides[1] = {ld_elems};
    const uint32_t box[2] = {box0, box1};
    return make_map(map, base, 2, dims, strides, box, mn_major);
}

// Map over packed 16-bit codes (plain 128-byte swizzle): rank 2 or 3, strides in elements.
int make_map16(CUtensorMap* map, const uint16_t* base, int rank, const uint64_t* dims, const uint64_t* strides_elems,
               const uint32_t* box) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) { set_last_cuda_error((int)cudaErrorSymbolNotFound); return QFMT_ERR_CUDA; }
    cuuint64_t d[3], st[2];
    cuuint32_t bx[3], estr[3] = {1, 1, 1};
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; bx[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) st[i] = strides_elems[i] * sizeof(uint16_t);
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, (cuuint32_t)rank, const_cast<uint16_t*>(base), d, st, bx, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_last_cuda_error(100000 + (int)r); return QFMT_ERR_CUDA; }
    return QFMT_OK;
}
// One operand of the packed contraction.  `extent` is its M (or N) size and `tile` the rows of it a
// CTA stages (128).  K-major: {K, extent} with 64 x tile boxes.  MN-major: 64-wide column blocks of
// 64 K rows; {64, K, extent / 64} with one box per stage when the extent is a multiple of 64
// (*blocked = 1), else the plain {extent, K} map, one 64 x 64 box per block, zero-filled past the end.
int make_operand_map16(CUtensorMap* map, const uint16_t* base, bool mn_major, uint64_t extent, uint64_t k, uint64_t ld,
                       uint32_t tile, int* blocked) {
    *blocked = 0;
    if (!mn_major) {
        const uint64_t dims[2] = {k, extent}, strides[1] = {ld};
        const uint32_t box[2] = {2 * kBK, tile};
        return make_map16(map, base, 2, dims, strides, box);
    }
    if (extent % 64 == 0) {
        *blocked = 1;
        const uint64_t dims[3] = {64, k, extent / 64}, strides[2] = {ld, 64};
        const uint32_t box[3] = {64, 2 * kBK, tile / 64};
        return make_map16(map, base, 3, dims, strides, box);
    }
    const uint64_t dims[2] = {extent, k}, strides[1] = {ld};
    const uint32_t box[2] = {64, 2 * kBK};
    return make_map16(map, base, 2, dims, strides, box);
}

// C (or the split-K partials) as a rank-3 map: [z][rows][N] with 32 x 32 x 1 boxes.
int make_map_c(CUtensorMap* map, float* base, uint64_t n, uint64_t rows, uint64_t zdim, uint64_t ld, uint64_t zstride) {
    const uint64_t dims[3] = {n, rows, zdim}, strides[2] = {ld, zstride};
    const uint32_t box[3] = {32, 32, 1};
    return make_map(map, base, 3, dims, strides, box, false);
}

// The same for N a multiple of 32, seen as [z][N / 32][rows][32]: a box takes kPOutBlocks whole 32 x 32
// blocks that are adjacent along the row, each landing in shared memory as one 4 KB swizzled block.
int make_map_c_blocked(CUtensorMap* map, float* base, uint64_t n, uint64_t rows, uint64_t zdim, uint64_t ld, uint64_t zstride) {
    const uint64_t dims[4] = {32, rows, n / 32, zdim}, strides[3] = {ld, 32, zstride};
    const uint32_t box[4] = {32, 32, (uint32_t)kPOutBlocks, 1};
    return make_map(map, base, 4, dims, strides, box, false);
}

// Sums the split-K partials [splits][rows][cols] (dense) into C in a fixed pairwise order: adjacent
// pairs level by level, an odd one out joining the next level as it is.  The tree is taken over
// kMax (a power of two >= splits) register slots with the absent ones holding -0, the value that
// changes no sum, so that every slot index is a compile-time constant.  T is float4 when rows can
// be moved 16 bytes at a time (cols then counts groups of four), else float.
__device__ __forceinline__ float tree_add(float a, float b) { return __fadd_rn(a, b); }
__device__ __forceinline__ float4 tree_add(float4 a, float4 b) {
    return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
}
__device__ __forceinline__ void tree_identity(float& v) { v = -0.0f; }
__device__ __forceinline__ void tree_identity(float4& v) { v = make_float4(-0.0f, -0.0f, -0.0f, -0.0f); }
template <typename T, int kMax>
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const T* __restrict__ part, T* __restrict__ C, long long rows, long long cols,
                     long long ldc, int splits) {
    grid_dependency_wait();   // the partial sums come from the kernel before this one
    grid_launch_dependents();
    const long long total = rows * cols;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        T v[kMax];
#pragma unroll
        for (int s = 0; s < kMax; ++s) {
            if (s < splits) v[s] = part[(long long)s * total + i];
            else tree_identity(v[s]);
        }
#pragma unroll
        for (int n = kMax; n > 1; n /= 2) {
#pragma unroll
            for (int s = 0; s < n / 2; ++s) v[s] = tree_add(v[2 * s], v[2 * s + 1]);
        }
        C[(i / cols) * ldc + (i % cols)] = v[0];
    }
}
template <typename T>
void launch_splitk_reduce_as(const float* part, float* C, long long rows, long long cols, long long ldc, int splits,
                             int sm_count, cudaStream_t stream) {
    const long long total = rows * cols, want = (total + 255) / 256, cap = (long long)sm_count * 16;
    const int blocks = (int)(want < cap ? want : cap);
    const T* p = reinterpret_cast<const T*>(part);
    T* c = reinterpret_cast<T*>(C);
    if (splits <= 2) (void)launch_overlapping(splitk_reduce_kernel<T, 2>, (unsigned)blocks, 256u, 0, stream, p, c, rows, cols, ldc, splits);
    else if (splits <= 4) (void)launch_overlapping(splitk_reduce_kernel<T, 4>, (unsigned)blocks, 256u, 0, stream, p, c, rows, cols, ldc, splits);
    else if (splits <= 8) (void)launch_overlapping(splitk_reduce_kernel<T, 8>, (unsigned)blocks, 256u, 0, stream, p, c, rows, cols, ldc, splits);
    else if (splits <= 16) (void)launch_overlapping(splitk_reduce_kernel<T, 16>, (unsigned)blocks, 256u, 0, stream, p, c, rows, cols, ldc, splits);
    else (void)launch_overlapping(splitk_reduce_kernel<T, 32>, (unsigned)blocks, 256u, 0, stream, p, c, rows, cols, ldc, splits);
}
// splits <= 32 (kMaxSplits).  The partials are dense, so groups of four stay inside a row when cols % 4 == 0.
void launch_splitk_reduce(const float* part, float* C, long long rows, long long cols, long long ldc, int splits,
                          int sm_count, cudaStream_t stream) {
    if (rows <= 0 || cols <= 0) return;
    const bool vec = cols % 4 == 0 && ldc % 4 == 0 && (reinterpret_cast<uintptr_t>(part) & 15) == 0 &&
                     (reinterpret_cast<uintptr_t>(C) & 15) == 0;
    if (vec) launch_splitk_reduce_as<float4>(part, C, rows, cols / 4, ldc / 4, splits, sm_count, stream);
    else launch_splitk_reduce_as<float>(part, C, rows, cols, ldc, splits, sm_count, stream);
}

constexpr size_t kWorkspaceHeader = 256;  // status area and padding ahead of the partial sums
// Tag of the next launch (GemmParams::launch_tag): process-wide, never zero, 48 bits.
unsigned long long next_launch_tag() {
    static std::atomic<unsigned long long> counter{0};
    return (counter.fetch_add(1) % ((1ull << 48) - 1)) + 1;
}
constexpr int kMaxSplits = 32;

// Balanced schedule, second pass: CTA b's first piece began inside a tile and sits in slot b; add it
// to the tile's place in C, which the CTA before wrote.  kFixupParts blocks per slot, each taking
// every kFixupParts-th row; N is a multiple of 32 here, so rows are moved as float4.
constexpr int kFixupParts = 16;
__global__ void __launch_bounds__(256)
streamk_fixup_kernel(const float* __restrict__ partials, float* __restrict__ C, int ctas, int num_tiles, int tiles_m,
                     int cpt, int tile_rows, long long M, long long N) {
    const int b = blockIdx.x / kFixupParts, part = blockIdx.x % kFixupParts;
    long long lo, hi;
    sk_range((long long)num_tiles * cpt, ctas, b, &lo, &hi);
    const long long tile = lo / cpt;
    if (lo >= hi || lo == tile * cpt) return;  // nothing, or the first piece began with its tile
    const long long tile_m = tile % tiles_m, tile_n = tile / tiles_m;
    const long long row0 = tile_m * tile_rows, col0 = tile_n * kBN;
    const long long rows = row0 + tile_rows < M ? tile_rows : M - row0;
    const long long cols4 = (col0 + kBN < N ? kBN : N - col0) / 4;
    const float* src = partials + (long long)b * tile_rows * N;  // the slot is addressed like [tile_rows][N]
    for (long long r = part; r < rows; r += kFixupParts) {
        for (long long c4 = threadIdx.x; c4 < cols4; c4 += blockDim.x) {
            float4* g = reinterpret_cast<float4*>(C + (row0 + r) * N + col0) + c4;
            const float4 a = *g, v = *(reinterpret_cast<const float4*>(src + r * N + col0) + c4);
            *g = make_float4(__fadd_rn(a.x, v.x), __fadd_rn(a.y, v.y), __fadd_rn(a.z, v.z), __fadd_rn(a.w, v.w));
        }
    }
}

int launch_gemm(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const CUtensorMap& mp,
                const RowMaps& rows, const GemmParams& p, const DeviceInfo& dev, cudaStream_t stream) {
    static bool attr_set[64] = {};
    if (dev.ordinal < 0 || dev.ordinal >= 64 || !attr_set[dev.ordinal]) {
        QFMT_CUDA_TRY(cudaFuncSetAttribute(gemm_tf32_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
        QFMT_CUDA_TRY(cudaFuncSetAttribute(gemm_tf32_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
        if (dev.ordinal >= 0 && dev.ordinal < 64) attr_set[dev.ordinal] = true;
    }
    const long long work = (long long)p.tiles_m * p.tiles_n * p.splits;
    const int grid = work < dev.sm_count ? (int)work : dev.sm_count;
    if (p.epi) QFMT_CUDA_TRY(launch_overlapping(gemm_tf32_kernel<true>, (unsigned)grid, (unsigned)kThreads, kSmemBytes, stream, ma, mb, mc, mp, rows, p));
    else QFMT_CUDA_TRY(launch_overlapping(gemm_tf32_kernel<false>, (unsigned)grid, (unsigned)kThreads, kSmemBytes, stream, ma, mb, mc, mp, rows, p));
    QFMT_CUDA_TRY(cudaGetLastError());
    if (p.sk_cpt > 0) {
        streamk_fixup_kernel<<<grid * kFixupParts, 64, 0, stream>>>(p.sk_partials, p.C, grid, p.tiles_m * p.tiles_n, p.tiles_m,
                                                       p.sk_cpt, p.tile_rows, (long long)p.M, (long long)p.N);
        QFMT_CUDA_TRY(cudaGetLastError());
    }
    return QFMT_OK;
}

void dense_defaults(GemmParams* p) {
    p->mode = 0;
    p->tile_rows = kBM;
    p->splits = 1;
    p->split_stride = 0;
    p->a_bytes = kABytes;
    p->b_bytes = kBBytes;
    p->img_rows = p->img_w = p->total_q = p->rows_per_blk = 1;
    p->taps = p->taps_s = p->cblocks = p->ck = 1;
    p->tap_sign = 1;
    p->off_h = p->off_w = 0;
    p->full_tiles_m = 0;
    p->conv_rows = 0;
    p->a_blocked = p->b_blocked = 0;
    p->c_blocked = 0;
    p->rows_box = 1;
    p->wg_segs = 1;
    p->wg_padded = 0;
    p->sk_cpt = 0;
    p->sk_pieces = 1;
    p->sk_partials = nullptr;
    p->sk_flags = nullptr;
    p->epi = 0;
    p->epi_rbias = nullptr;
    p->epi_stats = nullptr;
}

}  // namespace

// Which kernel a dense product runs on: 0 automatic, 1 single-CTA tiles (128 x 256), 2 CTA-pair
// tiles (256 x 256), 3 CTA-pair tiles under the balanced schedule wherever it applies.  Process-wide;
// see qfmt_gemm_tile_policy.
static std::atomic<int> g_tile_policy{0};

// Which kernel the forward / data-gradient products of a convolution run on: 0 automatic (CTA pairs
// when there are two or more M-tiles, the balanced schedule by estimated cost), 1 always the single-CTA
// kernel, 2 CTA pairs on whole tiles, 3 CTA pairs under the balanced schedule wherever it applies.
// See qfmt_gemm_tile_policy.
static std::atomic<int> g_conv_pair_policy{0};

// How a dense product is laid over the GPU: tile shape and split-K factor.
struct DensePlan {
    bool pair;
    int splits;
    bool sk;  // CTA-pair tiles under the balanced schedule (GemmParams::sk_flags)
};
constexpr int kPlanPairs = 74;  // CTA pairs of a 148-SM part: the balanced schedule is dealt among exactly these
constexpr size_t kSkFlagBytes = ((size_t)(kPlanPairs + 1) * 16 * sizeof(int) + 255) & ~(size_t)255;

// Picks the plan with the least estimated time.  The unit is the time one CTA pair needs for one
// 64-element K chunk of a 256 x 256 tile, about a microsecond; a single CTA needs 1.07 of it for
// half the area.  A tile costs its chunks plus three units of exposed epilogue; split K adds a
// reduction pass over (splits + 1) x M x N floats at about 6.5 TB/s (measured: the partials are still in L2) plus a launch.  The wave count
// is taken for a 148-SM part whatever the device, so that the plan, and with it the summation
// order, depends on the problem alone.
DensePlan plan_dense(int64_t M, int64_t N, int64_t K, int policy_override = -1) {
    const int chosen = g_tile_policy.load();
    const bool want_sk = chosen == 3;
    const int policy = policy_override >= 0 ? policy_override : (want_sk ? 2 : chosen);
    const int64_t kb_total = (K + kBK - 1) / kBK;
    DensePlan best = {policy == 2, 1, false};
    double best_cost = -1.0;
    for (int pair = 0; pair < 2; ++pair) {
        if (policy == 1 && pair) continue;
        if (policy == 2 && !pair) continue;
        if (policy == 0 && pair && M <= kBM) continue;  // with one row of tiles the second CTA of a pair would idle
        const int64_t tile_rows = pair ? 2 * kBM : kBM, units = pair ? 74 : 148;
        const int64_t tiles = ((M + tile_rows - 1) / tile_rows) * ((N + kBN - 1) / kBN);
        const double per_chunk = pair ? 1.0 : 1.07;
        for (int64_t want = 1; want <= kMaxSplits; ++want) {
            const int64_t per = (kb_total + want - 1) / want;           // K blocks per split
            if (want > 1 && per < 16) break;                            // at least 512 K elements per split
            const int64_t splits = per > 0 ? (kb_total + per - 1) / per : 1;
            if (splits != want) continue;                               // same plan as a smaller request
            const int64_t waves = (tiles * splits + units - 1) / units;
            double cost = (double)waves * ((double)((per + kChunkKB - 1) / kChunkKB) * per_chunk + 3.0);
            if (splits > 1) cost += 3.0 + (double)(splits + 1) * (double)M * (double)N * 4.0 / 6.5e6;
            if (best_cost < 0.0 || cost < best_cost * 0.97) {  // more splits only for a clear gain
                best_cost = cost;
                best = {pair != 0, (int)splits, false};
            }
        }
        // Balanced schedule: the tiles' chunks dealt among the 74 pairs in equal ranges.  A pair then runs
        // tiles / 74 + 1 pieces, each with its own move of sums to C.  Needs ranges of at least a tile.
        // Only on request (policy 3).  Measured on dense products it loses to whole tiles even where a
        // third of the last wave idles (8192 x 1024 x 1024: 48 against 40 us): pairs that walk through
        // different tiles at different K offsets share no operand bytes in flight, each pair has one more
        // move of sums to C, and the planner's automatic choice therefore never takes it.
        if (pair && want_sk && tiles >= kPlanPairs) {
            best = {true, 1, true};
            break;
        }
    }
    return best;
}

int launch_pair(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const GemmParams& p,
                const DeviceInfo& dev, cudaStream_t stream, int kind = kKindTf32) {
    static bool attr_set[64] = {};
    if (dev.ordinal < 0 || dev.ordinal >= 64 || !attr_set[dev.ordinal]) {
#define QFMT_PAIR_ATTR(...)                                                                                       \
    QFMT_CUDA_TRY(cudaFuncSetAttribute(gemm_tf32_pair_kernel<__VA_ARGS__>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                       (int)kPairSmemBytes))
        QFMT_PAIR_ATTR(false, kKindTf32, false);
        QFMT_PAIR_ATTR(false, kKindTf32, true);
        QFMT_PAIR_ATTR(true, kKindTf32, false);
        QFMT_PAIR_ATTR(false, kKindF16, false);
        QFMT_PAIR_ATTR(false, kKindF16, true);
        QFMT_PAIR_ATTR(false, kKindBf16, false);
        QFMT_PAIR_ATTR(false, kKindBf16, true);
#undef QFMT_PAIR_ATTR
        if (dev.ordinal >= 0 && dev.ordinal < 64) attr_set[dev.ordinal] = true;
    }
    const long long work = (long long)p.tiles_m * p.tiles_n * p.splits;
    const long long clusters = p.sk_flags != nullptr ? kPlanPairs : (work < dev.sm_count / 2 ? work : dev.sm_count / 2);
    const unsigned grid = (unsigned)(2 * clusters);
    const bool sk = p.sk_flags != nullptr;
#define QFMT_PAIR_LAUNCH(...) \
    QFMT_CUDA_TRY(launch_overlapping(gemm_tf32_pair_kernel<__VA_ARGS__>, grid, (unsigned)kThreads, kPairSmemBytes, stream, ma, mb, mc, p))
    if (kind == kKindF16) { if (sk) QFMT_PAIR_LAUNCH(false, kKindF16, true); else QFMT_PAIR_LAUNCH(false, kKindF16, false); }
    else if (kind == kKindBf16) { if (sk) QFMT_PAIR_LAUNCH(false, kKindBf16, true); else QFMT_PAIR_LAUNCH(false, kKindBf16, false); }
    else if (p.epi) QFMT_PAIR_LAUNCH(true, kKindTf32, false);
    else if (sk) QFMT_PAIR_LAUNCH(false, kKindTf32, true);
    else QFMT_PAIR_LAUNCH(false, kKindTf32, false);
#undef QFMT_PAIR_LAUNCH
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}

int launch_conv_pair(const CUtensorMap& mb, const CUtensorMap& mc, const CUtensorMap& mc2, const RowMaps& rows,
                     const GemmParams& p, const DeviceInfo& dev, cudaStream_t stream) {
    static bool attr_set[64] = {};
    if (dev.ordinal < 0 || dev.ordinal >= 64 || !attr_set[dev.ordinal]) {
        QFMT_CUDA_TRY(cudaFuncSetAttribute(gemm_conv_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)kPairSmemBytes));
        QFMT_CUDA_TRY(cudaFuncSetAttribute(gemm_conv_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)kPairSmemBytes));
        if (dev.ordinal >= 0 && dev.ordinal < 64) attr_set[dev.ordinal] = true;
    }
    const long long work = (long long)p.tiles_m * p.tiles_n;
    const long long clusters = p.sk_flags != nullptr ? kPlanPairs : (work < dev.sm_count / 2 ? work : dev.sm_count / 2);
    if (p.sk_flags != nullptr)
        QFMT_CUDA_TRY(launch_overlapping(gemm_conv_pair_kernel<true>, (unsigned)(2 * clusters), (unsigned)kThreads, kPairSmemBytes, stream,
                                         mb, mc, mc2, rows, p));
    else
        QFMT_CUDA_TRY(launch_overlapping(gemm_conv_pair_kernel<false>, (unsigned)(2 * clusters), (unsigned)kThreads, kPairSmemBytes, stream,
                                         mb, mc, mc2, rows, p));
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}

int launch_wgrad_pair(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const GemmParams& p,
                      const DeviceInfo& dev, cudaStream_t stream) {
    static bool attr_set[64] = {};
    if (dev.ordinal < 0 || dev.ordinal >= 64 || !attr_set[dev.ordinal]) {
        QFMT_CUDA_TRY(cudaFuncSetAttribute(gemm_wgrad_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)kPairSmemBytes));
        if (dev.ordinal >= 0 && dev.ordinal < 64) attr_set[dev.ordinal] = true;
    }
    const long long work = (long long)p.tiles_m * p.tiles_n * p.splits;
    const long long clusters = work < dev.sm_count / 2 ? work : dev.sm_count / 2;
    QFMT_CUDA_TRY(launch_overlapping(gemm_wgrad_pair_kernel, (unsigned)(2 * clusters), (unsigned)kThreads, kPairSmemBytes, stream, ma, mb, mc, p));
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}

// Layer-output epilogue request for gemm_device: the rounded, zero-padded bias and the record.
struct EpiArgs {
    const float* rbias;
    qfmt_stats_t* stats;
};
// The epilogue runs on the sums of one group held in registers: at most this many K elements.
constexpr int64_t kEpiMaxK = (int64_t)kFlushChunks * kChunkKB * kBK;

// Whether the balanced schedule can take a product of `tiles` pair tiles of `cpt` chunks: the chunk count
// stays in 32 bits and a pair's pieces fit the kernel's table.
bool pair_schedule_fits(long long tiles, long long cpt) {
    const long long total = tiles * cpt;
    if (cpt <= 0 || total >= (1ll << 30)) return false;
    const long long range = (total + kPlanPairs - 1) / kPlanPairs;
    return (range + cpt - 1) / cpt + 1 <= kMaxSkPieces;
}

// Turns the balanced schedule of the pair kernel on: chunks per tile, the most pieces a pair can have,
// and the flag words behind the workspace header (cleared on the stream).
int enable_pair_schedule(GemmParams* p, void* d_workspace, cudaStream_t stream) {
    p->sk_cpt = (p->kb_total + kChunkKB - 1) / kChunkKB;
    const long long total = (long long)p->tiles_m * p->tiles_n * p->sk_cpt;
    const long long range = (total + kPlanPairs - 1) / kPlanPairs;
    p->sk_pieces = (int)((range + p->sk_cpt - 1) / p->sk_cpt + 1);
    p->sk_q = (int)(total / kPlanPairs);
    p->sk_r = (int)(total % kPlanPairs);
    p->sk_flags = reinterpret_cast<int*>(reinterpret_cast<char*>(d_workspace) + kWorkspaceHeader);
    QFMT_CUDA_TRY(launch_overlapping(zero_words_kernel, 1u, 256u, 0, stream, p->sk_flags, (int)(kSkFlagBytes / sizeof(int))));
    return QFMT_OK;
}

// Host-side checks of a dense product's arguments, in the order the entry points report them: format,
// descriptors and shapes, workspace, output and operand pointers.  Touches no device state.  On
// QFMT_OK *M, *N, *K hold the product's dimensions (M or N may be zero: nothing to do).
int validate_gemm_args(const qfmt_matrix_t* A, const qfmt_matrix_t* B, const float* d_C, int64_t ldc,
                       const qfmt_format_t* fmt, const void* d_workspace, size_t workspace_bytes, int64_t* M_out,
                       int64_t* N_out, int64_t* K_out) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    if (fmt->m > 10) return QFMT_ERR_BAD_FORMAT;  // beyond TF32's mantissa: products would not be exact
    if (A == nullptr || B == nullptr) return QFMT_ERR_BAD_ARG;
    if (A->rows < 0 || A->cols < 0 || B->rows < 0 || B->cols < 0) return QFMT_ERR_BAD_ARG;
    const int64_t M = A->trans ? A->cols : A->rows, K = A->trans ? A->rows : A->cols;
    const int64_t Kb = B->trans ? B->cols : B->rows, N = B->trans ? B->rows : B->cols;
    if (K != Kb) return QFMT_ERR_BAD_ARG;
    if (M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return QFMT_ERR_BAD_ARG;
    if (A->ld < A->cols || B->ld < B->cols || ldc < N) return QFMT_ERR_BAD_ARG;
    if (d_workspace == nullptr || workspace_bytes < 16 || (reinterpret_cast<uintptr_t>(d_workspace) & 15u))
        return QFMT_ERR_BAD_ARG;
    *M_out = M; *N_out = N; *K_out = K;
    if (M == 0 || N == 0) return QFMT_OK;
    if (A->ptr == nullptr && K != 0) return QFMT_ERR_BAD_ARG;
    if (B->ptr == nullptr && K != 0) return QFMT_ERR_BAD_ARG;
    if (d_C == nullptr || (reinterpret_cast<uintptr_t>(d_C) & 3u)) return QFMT_ERR_BAD_ARG;
    // TMA needs 16-byte aligned bases and row pitches
    if ((reinterpret_cast<uintptr_t>(A->ptr) & 15u) || (reinterpret_cast<uintptr_t>(B->ptr) & 15u) ||
        (A->ld & 3) || (B->ld & 3))
        return QFMT_ERR_BAD_ARG;
    return QFMT_OK;
}

int gemm_device(const qfmt_matrix_t* A, const qfmt_matrix_t* B, float* d_C, int64_t ldc, const qfmt_format_t* fmt,
                void* d_workspace, size_t workspace_bytes, cudaStream_t stream, const EpiArgs* epi = nullptr) {
    int64_t M = 0, N = 0, K = 0;
    int rc = validate_gemm_args(A, B, d_C, ldc, fmt, d_workspace, workspace_bytes, &M, &N, &K);
    if (rc != QFMT_OK) return rc;
    if (M == 0 || N == 0) return QFMT_OK;
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;

    if (K == 0) {  // no kernel: the status area itself says "no error"
        QFMT_CUDA_TRY(cudaMemsetAsync(d_workspace, 0, 16, stream));
        QFMT_CUDA_TRY(cudaMemset2DAsync(d_C, (size_t)ldc * sizeof(float), 0, (size_t)N * sizeof(float), (size_t)M, stream));
        return QFMT_OK;
    }

    GemmParams p;
    dense_defaults(&p);
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    p.ldc = ldc;
    p.C = d_C;
    p.status = reinterpret_cast<unsigned long long*>(d_workspace);
    p.launch_tag = next_launch_tag();
    p.a_mn_major = A->trans ? 1 : 0;
    p.b_mn_major = B->trans ? 0 : 1;
    const DensePlan plan = plan_dense(M, N, K);
    const bool pair = plan.pair;
    p.tile_rows = pair ? 2 * kBM : kBM;
    p.tiles_m = (int)((M + p.tile_rows - 1) / p.tile_rows);
    p.tiles_n = (int)((N + kBN - 1) / kBN);
    p.kb_total = (int)((K + kBK - 1) / kBK);
    p.kb_per_split = p.kb_total;
    // TMA stores clip at 16-byte granularity along the row, so N must be a multiple of 4 as well.
    p.tma_store = ((reinterpret_cast<uintptr_t>(d_C) & 15u) == 0 && (ldc & 3) == 0 && (N & 3) == 0) ? 1 : 0;

    // Split K when the workspace the caller lent has room for the partial sums (the recommended size
    // from qfmt_gemm_workspace_bytes always has); a smaller workspace gets fewer splits.
    int splits = epi != nullptr ? 1 : plan.splits;
    // The balanced schedule needs every pair resident at once (148 SMs), room for its flags in the
    // workspace, and the blocked C map.
    const bool sk = plan.sk && epi == nullptr && pair && dev.sm_count >= 2 * kPlanPairs && p.tma_store &&
                    (N & 31) == 0 && workspace_bytes >= kWorkspaceHeader + kSkFlagBytes &&
                    pair_schedule_fits((long long)p.tiles_m * p.tiles_n, (p.kb_total + kChunkKB - 1) / kChunkKB);
    if (epi != nullptr) {
        if (K > kEpiMaxK || fmt->e > 6) return QFMT_ERR_BAD_ARG;  // callers check before asking
        qfmt_format_t f = *fmt;
        f.loss_scale = 1.0f;
        p.epi = 1;
        p.epi_rbias = epi->rbias;
        p.epi_stats = epi->stats;
        p.epi_q = make_params(f);
    }
    while (splits > 1 && kWorkspaceHeader + (size_t)splits * (size_t)M * (size_t)N * sizeof(float) > workspace_bytes) --splits;
    float* partials = reinterpret_cast<float*>(reinterpret_cast<char*>(d_workspace) + kWorkspaceHeader);
    if (sk) {
        rc = enable_pair_schedule(&p, d_workspace, stream);
        if (rc != QFMT_OK) return rc;
    } else if (splits > 1) {
        p.kb_per_split = (p.kb_total + splits - 1) / splits;
        p.splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;
        p.split_stride = (long long)M * N;
        p.C = partials;
        p.ldc = N;
        p.tma_store = (N & 3) == 0 ? 1 : 0;
    }

    CUtensorMap ma, mb, mc;
    // An MN-major operand is staged as 32-wide column blocks of 4 KB.  When its extent is a multiple
    // of 32 the matrix is described as {32, K, extent / 32} and one copy brings all of a stage's
    // blocks; otherwise the last block would reach past the row's end, and each block is copied by
    // itself from the plain rank-2 map, which zero-fills beyond the extent.
    p.a_blocked = (p.a_mn_major && (M & 31) == 0) ? 1 : 0;
    p.b_blocked = (p.b_mn_major && (N & 31) == 0) ? 1 : 0;
    if (p.a_blocked) {
        const uint64_t dims[3] = {32, (uint64_t)K, (uint64_t)M / 32}, strides[2] = {(uint64_t)A->ld, 32};
        const uint32_t box[3] = {32, kBK, kBM / 32};
        rc = make_map(&ma, A->ptr, 3, dims, strides, box, true);
    } else if (p.a_mn_major) rc = make_map_2d(&ma, A->ptr, (uint64_t)M, (uint64_t)K, (uint64_t)A->ld, 32, kBK, true);
    else rc = make_map_2d(&ma, A->ptr, (uint64_t)K, (uint64_t)M, (uint64_t)A->ld, kBK, kBM, false);
    if (rc != QFMT_OK) return rc;
    if (p.b_blocked) {
        const uint64_t dims[3] = {32, (uint64_t)K, (uint64_t)N / 32}, strides[2] = {(uint64_t)B->ld, 32};
        const uint32_t box[3] = {32, kBK, (uint32_t)((pair ? kBN / 2 : kBN) / 32)};
        rc = make_map(&mb, B->ptr, 3, dims, strides, box, true);
    } else if (p.b_mn_major) rc = make_map_2d(&mb, B->ptr, (uint64_t)N, (uint64_t)K, (uint64_t)B->ld, 32, kBK, true);
    else rc = make_map_2d(&mb, B->ptr, (uint64_t)K, (uint64_t)N, (uint64_t)B->ld, kBK, pair ? kBN / 2 : kBN, false);
    if (rc != QFMT_OK) return rc;
    p.c_blocked = (pair && p.tma_store && (N & 31) == 0) ? 1 : 0;
    if (p.c_blocked)
        rc = make_map_c_blocked(&mc, p.C, (uint64_t)N, (uint64_t)M, (uint64_t)p.splits, (uint64_t)p.ldc, (uint64_t)M * (uint64_t)p.ldc);
    else if (p.tma_store)
        rc = make_map_c(&mc, p.C, (uint64_t)N, (uint64_t)M, (uint64_t)p.splits, (uint64_t)p.ldc, (uint64_t)M * (uint64_t)p.ldc);
    else mc = ma;  // unused by the kernel
    if (rc != QFMT_OK) return rc;
    if (pair) {
        rc = launch_pair(ma, mb, mc, p, dev, stream);
    } else {
        RowMaps rows;
        for (int i = 0; i < kMaxRowMaps; ++i) rows.m[i] = ma;  // unused in dense mode
        rc = launch_gemm(ma, mb, mc, mc, rows, p, dev, stream);
    }
    if (rc != QFMT_OK) return rc;
    if (p.splits > 1) {
        launch_splitk_reduce(partials, d_C, M, N, ldc, p.splits, dev.sm_count, stream);
        QFMT_CUDA_TRY(cudaGetLastError());
    }
    return QFMT_OK;
}

// C = op(A) op(B) on packed 16-bit codes of 1/5/10 (binary16 words) or 1/8/7 (bfloat16 words): the
// pair kernel with kind::f16 MMAs.  A stage is 64 K elements per 128-byte row and a TMEM chunk 128
// (eight MMAs, as for TF32); the plan is the one of a TF32 product of half the length, which costs
// the same number of MMAs.
int gemm16_device(const qfmt_matrix16_t* A, const qfmt_matrix16_t* B, float* d_C, int64_t ldc, const qfmt_format_t* fmt,
                  void* d_workspace, size_t workspace_bytes, cudaStream_t stream) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    const bool f16 = fmt->e == 5 && fmt->m == 10, bf16 = fmt->e == 8 && fmt->m == 7;
    if (!f16 && !bf16) return QFMT_ERR_BAD_FORMAT;
    if (A == nullptr || B == nullptr) return QFMT_ERR_BAD_ARG;
    if (A->rows < 0 || A->cols < 0 || B->rows < 0 || B->cols < 0) return QFMT_ERR_BAD_ARG;
    const int64_t M = A->trans ? A->cols : A->rows, K = A->trans ? A->rows : A->cols;
    const int64_t Kb = B->trans ? B->cols : B->rows, N = B->trans ? B->rows : B->cols;
    if (K != Kb) return QFMT_ERR_BAD_ARG;
    if (M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return QFMT_ERR_BAD_ARG;
    if (A->ld < A->cols || B->ld < B->cols || ldc < N) return QFMT_ERR_BAD_ARG;
    if (d_workspace == nullptr || workspace_bytes < 16 || (reinterpret_cast<uintptr_t>(d_workspace) & 15u))
        return QFMT_ERR_BAD_ARG;
    if (M == 0 || N == 0) return QFMT_OK;
    if ((A->ptr == nullptr || B->ptr == nullptr) && K != 0) return QFMT_ERR_BAD_ARG;
    if (d_C == nullptr || (reinterpret_cast<uintptr_t>(d_C) & 3u)) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(A->ptr) & 15u) || (reinterpret_cast<uintptr_t>(B->ptr) & 15u) || (A->ld & 7) ||
        (B->ld & 7))
        return QFMT_ERR_BAD_ARG;  // TMA: 16-byte aligned bases and row pitches
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;
    if (K == 0) {
        QFMT_CUDA_TRY(cudaMemsetAsync(d_workspace, 0, 16, stream));
        QFMT_CUDA_TRY(cudaMemset2DAsync(d_C, (size_t)ldc * sizeof(float), 0, (size_t)N * sizeof(float), (size_t)M, stream));
        return QFMT_OK;
    }
    GemmParams p;
    dense_defaults(&p);
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    p.ldc = ldc;
    p.C = d_C;
    p.status = reinterpret_cast<unsigned long long*>(d_workspace);
    p.launch_tag = next_launch_tag();
    p.a_mn_major = A->trans ? 1 : 0;
    p.b_mn_major = B->trans ? 0 : 1;
    p.tile_rows = 2 * kBM;
    p.tiles_m = (int)((M + p.tile_rows - 1) / p.tile_rows);
    p.tiles_n = (int)((N + kBN - 1) / kBN);
    p.kb_total = (int)((K + 2 * kBK - 1) / (2 * kBK));
    p.kb_per_split = p.kb_total;
    p.tma_store = ((reinterpret_cast<uintptr_t>(d_C) & 15u) == 0 && (ldc & 3) == 0 && (N & 3) == 0) ? 1 : 0;
    const DensePlan plan = plan_dense(M, N, (K + 1) / 2, 2);
    int splits = plan.splits;
    const bool sk = plan.sk && dev.sm_count >= 2 * kPlanPairs && p.tma_store && (N & 31) == 0 &&
                    workspace_bytes >= kWorkspaceHeader + kSkFlagBytes &&
                    pair_schedule_fits((long long)p.tiles_m * p.tiles_n, (p.kb_total + kChunkKB - 1) / kChunkKB);
    while (splits > 1 && kWorkspaceHeader + (size_t)splits * (size_t)M * (size_t)N * sizeof(float) > workspace_bytes) --splits;
    float* partials = reinterpret_cast<float*>(reinterpret_cast<char*>(d_workspace) + kWorkspaceHeader);
    if (sk) {
        rc = enable_pair_schedule(&p, d_workspace, stream);
        if (rc != QFMT_OK) return rc;
    } else if (splits > 1) {
        p.kb_per_split = (p.kb_total + splits - 1) / splits;
        p.splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;
        p.split_stride = (long long)M * N;
        p.C = partials;
        p.ldc = N;
        p.tma_store = (N & 3) == 0 ? 1 : 0;
    }
    CUtensorMap ma, mb, mc;
    rc = make_operand_map16(&ma, A->ptr, p.a_mn_major != 0, (uint64_t)M, (uint64_t)K, (uint64_t)A->ld, kBM, &p.a_blocked);
    if (rc != QFMT_OK) return rc;
    rc = make_operand_map16(&mb, B->ptr, p.b_mn_major != 0, (uint64_t)N, (uint64_t)K, (uint64_t)B->ld, kBN / 2, &p.b_blocked);
    if (rc != QFMT_OK) return rc;
    p.c_blocked = (p.tma_store && (N & 31) == 0) ? 1 : 0;
    if (p.c_blocked)
        rc = make_map_c_blocked(&mc, p.C, (uint64_t)N, (uint64_t)M, (uint64_t)p.splits, (uint64_t)p.ldc, (uint64_t)M * (uint64_t)p.ldc);
    else if (p.tma_store)
        rc = make_map_c(&mc, p.C, (uint64_t)N, (uint64_t)M, (uint64_t)p.splits, (uint64_t)p.ldc, (uint64_t)M * (uint64_t)p.ldc);
    else mc = ma;  // unused by the kernel
    if (rc != QFMT_OK) return rc;
    rc = launch_pair(ma, mb, mc, p, dev, stream, f16 ? kKindF16 : kKindBf16);
    if (rc != QFMT_OK) return rc;
    if (p.splits > 1) {
        launch_splitk_reduce(partials, d_C, M, N, ldc, p.splits, dev.sm_count, stream);
        QFMT_CUDA_TRY(cudaGetLastError());
    }
    return QFMT_OK;
}

// ------------------------------------------------------------------------------------------------
// Convolution layers as implicit GEMMs on channels-last tensors (unit stride, zero padding).
// ------------------------------------------------------------------------------------------------
namespace {
struct ConvPlan {
    int64_t oh, ow;
    bool pair;       // forward / data gradient on CTA pairs (two M-tiles of whole image rows per pair)
    bool pair_sk;    // ... under the balanced schedule of the pair kernel
    bool pair_wgrad; // filter gradient on CTA pairs (padded stages, C_out of at least 256)
    int splits;
    int sk_cpt;      // forward / data gradient: chunks per tile when the balanced schedule is used, else 0
    int sk_pieces;
    size_t workspace;
};
// Output rows per K stage of the filter gradient, and whether stages are padded (GemmParams::wg_padded):
// padded when every stage then stays inside one image and a tile's 256 columns inside one tap.
int wgrad_rows_per_stage(int64_t oh, int64_t ow, int64_t c_in, int* padded_row) {
    int wpad = 1;
    while (wpad < ow) wpad *= 2;
    const bool padded = wpad <= kBK && oh % (kBK / wpad) == 0 && c_in % kBN == 0;
    if (padded_row != nullptr) *padded_row = padded ? wpad : 0;
    if (ow > kBK) return 1;
    return padded ? kBK / wpad : kBK / (int)ow;
}
// K stages per output row of the filter gradient: rows longer than a stage's 32 pixels are cut into 32-pixel pieces.
int wgrad_row_segments(int64_t ow) { return ow > kBK ? (int)((ow + kBK - 1) / kBK) : 1; }
constexpr int kPlanSms = 148;  // B200; the split factor is planned for it so that it does not vary
int plan_conv(int op, const qfmt_conv_t* g, ConvPlan* plan) {
    if (g == nullptr || op < QFMT_CONV_FWD || op > QFMT_CONV_WGRAD) return QFMT_ERR_BAD_ARG;
    if (g->n <= 0 || g->c_in <= 0 || g->h <= 0 || g->w <= 0 || g->c_out <= 0 || g->r <= 0 || g->s <= 0 ||
        g->pad_h < 0 || g->pad_w < 0)
        return QFMT_ERR_BAD_ARG;
    if ((g->c_in & 31) || (g->c_out & 31)) return QFMT_ERR_BAD_ARG;  // 32-channel blocks must not straddle taps
    plan->oh = (int64_t)g->h + 2 * g->pad_h - g->r + 1;
    plan->ow = (int64_t)g->w + 2 * g->pad_w - g->s + 1;
    if (plan->oh <= 0 || plan->ow <= 0) return QFMT_ERR_BAD_ARG;
    if ((int64_t)g->n * g->h * g->w > (1 << 30) || (int64_t)g->n * plan->oh * plan->ow > (1 << 30) ||
        (int64_t)g->r * g->s * g->c_in > (1 << 30))
        return QFMT_ERR_BAD_ARG;
    plan->splits = 1;
    plan->pair = false;
    plan->pair_sk = false;
    plan->pair_wgrad = false;
    plan->sk_cpt = 0;
    plan->sk_pieces = 1;
    plan->workspace = kWorkspaceHeader;
    if (g->r == 1 && g->s == 1 && g->pad_h == 0 && g->pad_w == 0) {
        // runs as a dense product (see conv_device): the dense planner's workspace, no row-length limits
        const int64_t pixels = (int64_t)g->n * g->h * g->w;
        const int64_t M = op == QFMT_CONV_WGRAD ? g->c_out : pixels;
        const int64_t N = op == QFMT_CONV_FWD ? g->c_out : g->c_in;
        const int64_t K = op == QFMT_CONV_FWD ? g->c_in : (op == QFMT_CONV_DGRAD ? g->c_out : pixels);
        const DensePlan dense = plan_dense(M, N, K);
        if (dense.sk) plan->workspace += kSkFlagBytes;
        else if (dense.splits > 1) plan->workspace += (size_t)dense.splits * (size_t)M * (size_t)N * sizeof(float);
        return QFMT_OK;
    }
    if (op == QFMT_CONV_FWD && plan->ow > kBM) return QFMT_ERR_BAD_ARG;   // an M-tile is made of whole output rows
    if (op == QFMT_CONV_DGRAD && g->w > kBM) return QFMT_ERR_BAD_ARG;
    if (op != QFMT_CONV_WGRAD) {
        // With more tiles than SMs and a last wave that leaves many SMs idle, the K chunks of all
        // tiles are dealt out in equal ranges instead (see GemmParams::sk_cpt).
        const bool fwd = op == QFMT_CONV_FWD;
        const int64_t rows = fwd ? plan->oh : g->h, width = fwd ? plan->ow : g->w;
        const int64_t rows_per_blk = kBM / width, n_cols = fwd ? g->c_out : g->c_in, src_c = fwd ? g->c_in : g->c_out;
        const int64_t tiles = (((int64_t)g->n * rows + rows_per_blk - 1) / rows_per_blk) * ((n_cols + kBN - 1) / kBN);
        const int64_t kb_total = (int64_t)g->r * g->s * (src_c / 32), cpt = (kb_total + kChunkKB - 1) / kChunkKB;
        const int64_t waves = (tiles + kPlanSms - 1) / kPlanSms;
        // Two or more M-tiles: CTA pairs, each CTA one M-tile and half of the filter columns (8 KB of
        // operands per MMA and CTA instead of 12).  The balanced schedule is priced as for dense products.
        const int64_t conv_tiles_m = ((int64_t)g->n * rows + rows_per_blk - 1) / rows_per_blk;
        if (conv_tiles_m >= 2 && g_conv_pair_policy.load() != 1) {
            plan->pair = true;
            const int64_t ptiles = ((conv_tiles_m + 1) / 2) * ((n_cols + kBN - 1) / kBN);
            if (ptiles >= kPlanPairs) {
                const int64_t pwaves = (ptiles + kPlanPairs - 1) / kPlanPairs;
                const double plain = (double)pwaves * ((double)cpt + 3.0);
                const double sk = (double)ptiles * (double)cpt / kPlanPairs + 3.0 * ((double)ptiles / kPlanPairs + 1.0);
                const int cp = g_conv_pair_policy.load();
                plan->pair_sk = cp == 3 || (cp == 0 && sk < plain * 0.97 && ptiles * cpt < (1ll << 30));
            }
            plan->workspace += kSkFlagBytes;
            return QFMT_OK;
        }
        // It pays when the last of a few waves is poorly filled and tiles are long: every piece ends
        // with an output flush of its own, and pieces that begin inside a tile are added to C later.
        if (tiles >= kPlanSms && waves <= 3 && waves * kPlanSms * 100 >= tiles * 115 && cpt >= 24) {
            const int64_t range = (tiles * cpt + kPlanSms - 1) / kPlanSms;
            plan->sk_cpt = (int)cpt;
            plan->sk_pieces = (int)((range + cpt - 1) / cpt + 1);
            plan->workspace += (size_t)kPlanSms * (size_t)(rows_per_blk * width) * (size_t)n_cols * sizeof(float);
        }
    }
    if (op == QFMT_CONV_WGRAD) {
        int padded_row = 0;
        const int rows_per_blk = wgrad_rows_per_stage(plan->oh, plan->ow, g->c_in, &padded_row);
        const int64_t kb_total = (((int64_t)g->n * plan->oh + rows_per_blk - 1) / rows_per_blk) * wgrad_row_segments(plan->ow);
        // CTA pairs (each CTA 128 rows of C_out and 128 columns of a tap) when the stages are padded, so that
        // one copy per operand fills a stage, and C_out fills a pair's 256 rows
        plan->pair_wgrad = padded_row > 0 && g->c_out >= 2 * kBM && g_conv_pair_policy.load() != 1;
        const int64_t tile_rows = plan->pair_wgrad ? 2 * kBM : kBM, units = plan->pair_wgrad ? kPlanPairs : kPlanSms;
        const int64_t tiles = (((int64_t)g->c_out + tile_rows - 1) / tile_rows) * (((int64_t)g->r * g->s * g->c_in + kBN - 1) / kBN);
        int64_t splits = units / tiles;
        if (splits > kMaxSplits) splits = kMaxSplits;
        if (splits > kb_total / 8) splits = kb_total / 8;   // at least eight stages per split
        if (splits < 1) splits = 1;
        const int64_t per = (kb_total + splits - 1) / splits;
        plan->splits = (int)((kb_total + per - 1) / per);
        if (plan->splits > 1)
            plan->workspace += (size_t)plan->splits * (size_t)g->c_out * (size_t)g->r * g->s * g->c_in * sizeof(float);
    }
    return QFMT_OK;
}
}  // namespace

namespace {
// A 1 x 1 filter without padding is a plain matrix product on channels-last tensors:
//   forward  Y[pixels][c_out]  = X[pixels][c_in] . W[c_out][c_in]^T
//   dgrad    dX[pixels][c_in]  = dY[pixels][c_out] . W[c_out][c_in]
//   wgrad    dW[c_out][c_in]   = dY[pixels][c_out]^T . X[pixels][c_in]
// so it runs on the dense kernels (CTA pairs, split K) instead of the implicit-GEMM modes.
bool conv_is_pointwise(const qfmt_conv_t* g) { return g->r == 1 && g->s == 1 && g->pad_h == 0 && g->pad_w == 0; }
void pointwise_operands(int op, const qfmt_conv_t* g, const float* d_p, const float* d_q, qfmt_matrix_t* A,
                        qfmt_matrix_t* B, int64_t* ldc) {
    const int64_t pixels = (int64_t)g->n * g->h * g->w;
    if (op == QFMT_CONV_FWD) {
        *A = {d_p, pixels, g->c_in, g->c_in, 0};
        *B = {d_q, g->c_out, g->c_in, g->c_in, 1};
        *ldc = g->c_out;
    } else if (op == QFMT_CONV_DGRAD) {
        *A = {d_p, pixels, g->c_out, g->c_out, 0};
        *B = {d_q, g->c_out, g->c_in, g->c_in, 0};
        *ldc = g->c_in;
    } else {
        *A = {d_p, pixels, g->c_out, g->c_out, 1};
        *B = {d_q, pixels, g->c_in, g->c_in, 0};
        *ldc = g->c_in;
    }
}
}  // namespace

int conv_device(int op, const qfmt_conv_t* g, const float* d_p, const float* d_q, float* d_out,
                const qfmt_format_t* fmt, void* d_workspace, size_t workspace_bytes, cudaStream_t stream) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    if (fmt->m > 10) return QFMT_ERR_BAD_FORMAT;
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;
    ConvPlan plan;
    rc = plan_conv(op, g, &plan);
    if (rc != QFMT_OK) return rc;
    if (d_p == nullptr || d_q == nullptr || d_out == nullptr) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_p) & 15u) || (reinterpret_cast<uintptr_t>(d_q) & 15u) ||
        (reinterpret_cast<uintptr_t>(d_out) & 15u))
        return QFMT_ERR_BAD_ARG;
    if (d_workspace == nullptr || workspace_bytes < plan.workspace || (reinterpret_cast<uintptr_t>(d_workspace) & 15u))
        return QFMT_ERR_BAD_ARG;
    if (conv_is_pointwise(g)) {
        qfmt_matrix_t A, B;
        int64_t ldc;
        pointwise_operands(op, g, d_p, d_q, &A, &B, &ldc);
        return gemm_device(&A, &B, d_out, ldc, fmt, d_workspace, workspace_bytes, stream);
    }
    const uint64_t N = g->n, CI = g->c_in, H = g->h, W = g->w, CO = g->c_out, R = g->r, S = g->s;
    const uint64_t OH = plan.oh, OW = plan.ow, TAPS = R * S;
    GemmParams p;
    dense_defaults(&p);
    p.status = reinterpret_cast<unsigned long long*>(d_workspace);
    p.launch_tag = next_launch_tag();
    p.taps = (int)TAPS;
    p.taps_s = (int)S;
    p.tma_store = 1;  // channel counts are multiples of 32 and the bases 16-byte aligned
    CUtensorMap ma, mb, mc;

    if (op == QFMT_CONV_FWD || op == QFMT_CONV_DGRAD) {
        const bool fwd = op == QFMT_CONV_FWD;
        // pixel space that is tiled: the output of the product
        const uint64_t rows = fwd ? OH : H, width = fwd ? OW : W;
        // activation-like operand that is read: X [N][H][W][CI] forward, dY [N][OH][OW][CO] data gradient
        const uint64_t src_h = fwd ? H : OH, src_w = fwd ? W : OW, src_c = fwd ? CI : CO;
        const uint64_t n_cols = fwd ? CO : CI;
        p.mode = 1;
        p.img_rows = (int)rows;
        p.img_w = (int)width;
        p.total_q = (int)(N * rows);
        p.rows_per_blk = kBM / (int)width;
        p.tile_rows = p.rows_per_blk * (int)width;
        p.M = (int)(N * rows * width);
        p.N = (int)n_cols;
        p.K = (int)(TAPS * src_c);
        p.ldc = (long long)n_cols;
        p.C = d_out;
        p.ck = (int)src_c;
        p.cblocks = (int)(src_c / 32);
        p.kb_total = (int)TAPS * p.cblocks;
        p.kb_per_split = p.kb_total;
        p.tap_sign = fwd ? 1 : -1;
        p.off_h = fwd ? -g->pad_h : g->pad_h;
        p.off_w = fwd ? -g->pad_w : g->pad_w;
        p.tiles_m = (p.total_q + p.rows_per_blk - 1) / p.rows_per_blk;
        p.tiles_n = (int)((n_cols + kBN - 1) / kBN);
        p.full_tiles_m = p.total_q / p.rows_per_blk;
        p.a_mn_major = 0;
        p.b_mn_major = fwd ? 0 : 1;
        p.a_bytes = (uint32_t)(p.tile_rows * 128);
        p.b_bytes = kBBytes;
        RowMaps rmaps;
        for (int cnt = 1; cnt <= kMaxRowMaps; ++cnt) {
            const uint64_t dims[4] = {src_c, src_w, src_h, N}, st[3] = {src_c, src_w * src_c, src_h * src_w * src_c};
            const uint32_t rows_in_box = cnt <= p.rows_per_blk ? (uint32_t)cnt : 1u;  // larger counts are never used
            const uint32_t box[4] = {32, (uint32_t)width, rows_in_box, 1};
            rc = make_map(&rmaps.m[cnt - 1], d_p, 4, dims, st, box, false);
            if (rc != QFMT_OK) return rc;
        }
        ma = rmaps.m[0];
        if (plan.pair) {
            // CTA pairs: a pair tile is two M-tiles; each CTA stages its own pixels and 128 filter columns
            const int conv_tiles_m = p.tiles_m;
            p.conv_rows = p.tile_rows;
            p.tile_rows = 2 * p.conv_rows;
            p.tiles_m = (conv_tiles_m + 1) / 2;
            p.c_blocked = 1;
            if (fwd) {
                rc = make_map_2d(&mb, d_q, TAPS * CI, CO, TAPS * CI, kBK, kBN / 2, false);
            } else {
                const uint64_t dims[4] = {32, TAPS, CO, CI / 32}, st[3] = {CI, TAPS * CI, 32};
                const uint32_t box[4] = {32, 1, kBK, (kBN / 2) / 32};
                rc = make_map(&mb, d_q, 4, dims, st, box, true);
            }
            if (rc != QFMT_OK) return rc;
            // C per M-tile: {32, conv_rows, N / 32, complete tiles}; the incomplete last tile has a map of its own
            CUtensorMap mc2;
            const uint64_t full = (uint64_t)p.full_tiles_m, rem = (uint64_t)p.M - full * (uint64_t)p.conv_rows;
            const uint32_t cbox[4] = {32, 32, (uint32_t)kPOutBlocks, 1};
            if (rem > 0) {
                const uint64_t d2[4] = {32, rem, n_cols / 32, 1}, s2[3] = {n_cols, 32, rem * n_cols};
                rc = make_map(&mc2, d_out + full * (uint64_t)p.conv_rows * n_cols, 4, d2, s2, cbox, false);
                if (rc != QFMT_OK) return rc;
            }
            if (full > 0) {
                const uint64_t d1[4] = {32, (uint64_t)p.conv_rows, n_cols / 32, full};
                const uint64_t s1[3] = {n_cols, 32, (uint64_t)p.conv_rows * n_cols};
                rc = make_map(&mc, d_out, 4, d1, s1, cbox, false);
                if (rc != QFMT_OK) return rc;
            } else {
                mc = mc2;
            }
            if (rem == 0) mc2 = mc;
            if (plan.pair_sk && dev.sm_count >= 2 * kPlanPairs &&
                pair_schedule_fits((long long)p.tiles_m * p.tiles_n, (p.kb_total + kChunkKB - 1) / kChunkKB)) {
                rc = enable_pair_schedule(&p, d_workspace, stream);
                if (rc != QFMT_OK) return rc;
            }
            return launch_conv_pair(mb, mc, mc2, rmaps, p, dev, stream);
        }
        if (fwd) {  // filters [CO][TAPS*CI], K contiguous
            rc = make_map_2d(&mb, d_q, TAPS * CI, CO, TAPS * CI, kBK, kBN, false);
        } else {    // filters [CO][TAPS][CI]: N = CI contiguous, K = CO rows
            const uint64_t dims[4] = {32, TAPS, CO, CI / 32}, st[3] = {CI, TAPS * CI, 32};
            const uint32_t box[4] = {32, 1, kBK, kBN / 32};
            rc = make_map(&mb, d_q, 4, dims, st, box, true);
        }
        if (rc != QFMT_OK) return rc;
        if (p.full_tiles_m > 0)
            rc = make_map_c(&mc, d_out, n_cols, (uint64_t)p.tile_rows, (uint64_t)p.full_tiles_m, n_cols,
                            (uint64_t)p.tile_rows * n_cols);
        else { mc = ma; p.tma_store = 0; }
        if (rc != QFMT_OK) return rc;
        CUtensorMap mp = mc;
        if (plan.sk_cpt > 0 && dev.sm_count == kPlanSms && p.tma_store) {  // the slots were sized for this many CTAs
            p.sk_cpt = plan.sk_cpt;
            p.sk_pieces = plan.sk_pieces;
            p.sk_partials = reinterpret_cast<float*>(reinterpret_cast<char*>(d_workspace) + kWorkspaceHeader);
            rc = make_map_c(&mp, p.sk_partials, n_cols, (uint64_t)p.tile_rows, (uint64_t)kPlanSms, n_cols,
                            (uint64_t)p.tile_rows * n_cols);
            if (rc != QFMT_OK) return rc;
        }
        return launch_gemm(ma, mb, mc, mp, rmaps, p, dev, stream);
    }

    // ---- filter gradient: dW [CO][TAPS*CI] = sum over pixels of dY^T (CO x pixels) * X_tap (pixels x CI)
    p.mode = 2;
    p.img_rows = (int)OH;
    p.img_w = (int)OW;
    p.total_q = (int)(N * OH);
    int padded_row = 0;
    p.rows_per_blk = wgrad_rows_per_stage((int64_t)OH, (int64_t)OW, (int64_t)CI, &padded_row);
    p.wg_padded = padded_row > 0 ? 1 : 0;
    const uint32_t wpad = (uint32_t)padded_row;
    p.M = (int)CO;
    p.N = (int)(TAPS * CI);
    p.K = (int)(N * OH * OW);
    p.ck = (int)CI;
    p.off_h = -g->pad_h;
    p.off_w = -g->pad_w;
    const bool pair_wgrad = plan.pair_wgrad && p.wg_padded;
    p.tile_rows = pair_wgrad ? 2 * kBM : kBM;
    p.tiles_m = (int)((CO + p.tile_rows - 1) / p.tile_rows);
    p.tiles_n = (p.N + kBN - 1) / kBN;
    p.wg_segs = wgrad_row_segments((int64_t)OW);
    p.kb_total = ((p.total_q + p.rows_per_blk - 1) / p.rows_per_blk) * p.wg_segs;
    p.splits = plan.splits;
    p.kb_per_split = (p.kb_total + p.splits - 1) / p.splits;
    p.a_mn_major = 1;
    p.b_mn_major = 1;
    // pixels a copy brings per image row: the whole row, or a 32-pixel piece of a longer one (zero-filled past its end)
    const uint32_t box_w = p.wg_segs > 1 ? (uint32_t)kBK : (uint32_t)OW;
    p.a_bytes = p.wg_padded ? kABytes : (uint32_t)(kBM / 32) * (uint32_t)p.rows_per_blk * box_w * 128u;
    p.b_bytes = p.wg_padded ? kBBytes : (uint32_t)(kBN / 32) * (uint32_t)p.rows_per_blk * box_w * 128u;
    float* partials = reinterpret_cast<float*>(reinterpret_cast<char*>(d_workspace) + kWorkspaceHeader);
    p.ldc = (long long)p.N;
    p.C = p.splits > 1 ? partials : d_out;
    p.split_stride = (long long)p.M * p.N;
    // a stage's image rows never straddle two images when their count divides the image height: one
    // copy then brings all of them for a channel block, else each row is copied by itself
    p.rows_box = (OH % p.rows_per_blk == 0) ? p.rows_per_blk : 1;
    if (p.wg_padded) {
        const uint64_t da[5] = {32, OW, OH, N, CO / 32}, sa_[4] = {CO, OW * CO, OH * OW * CO, 32};
        const uint32_t ba[5] = {32, wpad, (uint32_t)p.rows_per_blk, 1, kBM / 32};
        rc = make_map(&ma, d_p, 5, da, sa_, ba, true);
        if (rc != QFMT_OK) return rc;
        const uint64_t db[5] = {32, W, H, N, CI / 32}, sb_[4] = {CI, W * CI, H * W * CI, 32};
        const uint32_t bb[5] = {32, wpad, (uint32_t)p.rows_per_blk, 1, (uint32_t)((pair_wgrad ? kBN / 2 : kBN) / 32)};
        rc = make_map(&mb, d_q, 5, db, sb_, bb, true);
        if (rc != QFMT_OK) return rc;
    } else {
    {
        const uint64_t dims[4] = {CO, OW, OH, N}, st[3] = {CO, OW * CO, OH * OW * CO};
        const uint32_t box[4] = {32, box_w, (uint32_t)p.rows_box, 1};
        rc = make_map(&ma, d_p, 4, dims, st, box, true);
        if (rc != QFMT_OK) return rc;
    }
    {
        const uint64_t dims[4] = {CI, W, H, N}, st[3] = {CI, W * CI, H * W * CI};
        const uint32_t box[4] = {32, box_w, (uint32_t)p.rows_box, 1};
        rc = make_map(&mb, d_q, 4, dims, st, box, true);
        if (rc != QFMT_OK) return rc;
    }
    }
    if (pair_wgrad) {
        p.c_blocked = 1;  // N = taps * C_in is a multiple of 32
        rc = make_map_c_blocked(&mc, p.C, (uint64_t)p.N, (uint64_t)p.M, (uint64_t)p.splits, (uint64_t)p.N, (uint64_t)p.M * p.N);
        if (rc != QFMT_OK) return rc;
        rc = launch_wgrad_pair(ma, mb, mc, p, dev, stream);
    } else {
        rc = make_map_c(&mc, p.C, (uint64_t)p.N, (uint64_t)p.M, (uint64_t)p.splits, (uint64_t)p.N, (uint64_t)p.M * p.N);
        if (rc != QFMT_OK) return rc;
        RowMaps rows;
        for (int i = 0; i < kMaxRowMaps; ++i) rows.m[i] = ma;  // unused by the filter gradient
        rc = launch_gemm(ma, mb, mc, mc, rows, p, dev, stream);
    }
    if (rc != QFMT_OK) return rc;
    if (p.splits > 1) {
        launch_splitk_reduce(partials, d_out, p.M, p.N, p.N, p.splits, dev.sm_count, stream);
        QFMT_CUDA_TRY(cudaGetLastError());
    }
    return QFMT_OK;
}

}  // namespace qfmt

extern "C" int qfmt_gemm(const qfmt_matrix_t* A, const qfmt_matrix_t* B, float* d_C, int64_t ldc,
                         const qfmt_format_t* fmt, void* d_workspace, size_t workspace_bytes, void* stream) {
    return qfmt::gemm_device(A, B, d_C, ldc, fmt, d_workspace, workspace_bytes, (cudaStream_t)stream);
}

extern "C" int qfmt_gemm_packed16(const qfmt_matrix16_t* A, const qfmt_matrix16_t* B, float* d_C, int64_t ldc,
                                  const qfmt_format_t* fmt, void* d_workspace, size_t workspace_bytes, void* stream) {
    return qfmt::gemm16_device(A, B, d_C, ldc, fmt, d_workspace, workspace_bytes, (cudaStream_t)stream);
}

extern "C" int qfmt_conv(int32_t op, const qfmt_conv_t* geom, const float* d_p, const float* d_q, float* d_out,
                         const qfmt_format_t* fmt, void* d_workspace, size_t workspace_bytes, void* stream) {
    return qfmt::conv_device(op, geom, d_p, d_q, d_out, fmt, d_workspace, workspace_bytes, (cudaStream_t)stream);
}

extern "C" size_t qfmt_conv_workspace_bytes(int32_t op, const qfmt_conv_t* geom) {
    qfmt::ConvPlan plan;
    if (qfmt::plan_conv(op, geom, &plan) != QFMT_OK) return 0;
    return plan.workspace;
}

namespace qfmt {
int bias_quantize_stats_device(const float* d_acc, int64_t ld_acc, const float* d_bias, void* d_out, int64_t ld_out,
                               int64_t rows, int64_t cols, const qfmt_format_t* fmt, qfmt_stats_t* d_stats,
                               int accumulate, cudaStream_t stream, bool pack);
namespace {

// Rounds the bias vector for the fused epilogue; entries n .. padded-1 become zero.
__global__ void __launch_bounds__(256)
round_bias_kernel(const float* __restrict__ bias, float* __restrict__ out, int n, int padded, QuantParams q) {
    const uint32_t inf_bits = (uint32_t)(q.top + q.code_off) << 23;
    for (int i = blockIdx.x * 256 + threadIdx.x; i < padded; i += gridDim.x * 256)
        out[i] = i < n ? __uint_as_float(round_value<false>(__float_as_uint(bias[i]), q, inf_bits)) : 0.0f;
}

size_t linear_bias_bytes(int64_t N) {  // rounded bias, padded with zeros to whole tiles
    return (size_t)((N + kBN - 1) / kBN) * kBN * sizeof(float);
}

}  // namespace

// 0 automatic, 1 epilogue inside the GEMM kernel whenever it applies, 2 always two kernels; see
// qfmt_linear_fusion_policy.
static std::atomic<int> g_fusion_policy{0};

int linear_forward_device(const qfmt_matrix_t* A, const qfmt_matrix_t* B, const float* d_bias, float* d_Y, int64_t ldy,
                          const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate, void* d_workspace,
                          size_t workspace_bytes, cudaStream_t stream) {
    int rc = validate_format(fmt);
    if (rc != QFMT_OK) return rc;
    if (fmt->m > 10 || fmt->loss_scale != 1.0f) return QFMT_ERR_BAD_FORMAT;
    if (A == nullptr || B == nullptr || d_bias == nullptr) return QFMT_ERR_BAD_ARG;
    if (accumulate != 0 && accumulate != 1) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_bias) & 3u) || (reinterpret_cast<uintptr_t>(d_stats) & 7u)) return QFMT_ERR_BAD_ARG;
    if (A->rows < 0 || A->cols < 0 || B->rows < 0 || B->cols < 0) return QFMT_ERR_BAD_ARG;
    const int64_t M = A->trans ? A->cols : A->rows, K = A->trans ? A->rows : A->cols;
    const int64_t N = B->trans ? B->rows : B->cols;
    if (M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return QFMT_ERR_BAD_ARG;
    if (d_workspace == nullptr || (reinterpret_cast<uintptr_t>(d_workspace) & 15u)) return QFMT_ERR_BAD_ARG;
    const size_t bias_bytes = linear_bias_bytes(N);
    if (workspace_bytes < kWorkspaceHeader + bias_bytes + 256) return QFMT_ERR_BAD_ARG;
    // layout: [status area and padding | GEMM partial sums (unfused path) ... | rounded bias at the end,
    // on a 256-byte boundary]
    const size_t gemm_bytes = (workspace_bytes - bias_bytes) & ~(size_t)255u;
    float* rbias = reinterpret_cast<float*>(reinterpret_cast<char*>(d_workspace) + gemm_bytes);
    // e <= 6: at most 128 bins.  Automatic means two kernels: measured on B200, the epilogue's ALU work
    // in the eight accumulate warps holds a tile longer than the separate full-occupancy pass costs.
    const bool fused = g_fusion_policy.load() == 1 && fmt->e <= 6 && K >= 1 && K <= kEpiMaxK && M > 0 && N > 0;
    if (!fused) {
        rc = gemm_device(A, B, d_Y, ldy, fmt, d_workspace, gemm_bytes, stream);
        if (rc != QFMT_OK) return rc;
        return bias_quantize_stats_device(d_Y, ldy, d_bias, d_Y, ldy, M, N, fmt, d_stats, accumulate, stream, false);
    }
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;
    if (d_stats != nullptr && accumulate == 0) QFMT_CUDA_TRY(cudaMemsetAsync(d_stats, 0, sizeof(qfmt_stats_t), stream));
    const int padded = (int)(((N + kBN - 1) / kBN) * kBN);
    round_bias_kernel<<<(padded + 255) / 256, 256, 0, stream>>>(d_bias, rbias, (int)N, padded, make_params(*fmt));
    QFMT_CUDA_TRY(cudaGetLastError());
    const EpiArgs epi = {rbias, d_stats};
    return gemm_device(A, B, d_Y, ldy, fmt, d_workspace, gemm_bytes, stream, &epi);
}

}  // namespace qfmt

extern "C" int qfmt_linear_forward(const qfmt_matrix_t* A, const qfmt_matrix_t* B, const float* d_bias, float* d_Y,
                                   int64_t ldy, const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate,
                                   void* d_workspace, size_t workspace_bytes, void* stream) {
    return qfmt::linear_forward_device(A, B, d_bias, d_Y, ldy, fmt, d_stats, accumulate, d_workspace, workspace_bytes,
                                       (cudaStream_t)stream);
}

extern "C" int qfmt_linear_fusion_policy(int policy) {
    if (policy < 0 || policy > 2) return QFMT_ERR_BAD_ARG;
    qfmt::g_fusion_policy.store(policy);
    return QFMT_OK;
}

extern "C" size_t qfmt_linear_forward_workspace_bytes(const qfmt_matrix_t* A, const qfmt_matrix_t* B) {
    if (A == nullptr || B == nullptr) return 0;
    const int64_t N = B->trans ? B->rows : B->cols;
    if (N < 0 || N > (1 << 30)) return 0;
    return qfmt_gemm_workspace_bytes(A, B) + qfmt::linear_bias_bytes(N) + 256;
}

extern "C" int qfmt_conv_tile_policy(int policy) {
    if (policy < 0 || policy > 3) return QFMT_ERR_BAD_ARG;
    qfmt::g_conv_pair_policy.store(policy);
    return QFMT_OK;
}

extern "C" int qfmt_selftest_pair_schedule(int64_t tiles, int32_t chunks_per_tile, int32_t pair, int32_t j, int32_t* out) {
    if (out == nullptr || tiles < qfmt::kPlanPairs || chunks_per_tile <= 0 || pair < 0 || pair >= qfmt::kPlanPairs || j < 0)
        return QFMT_ERR_BAD_ARG;
    if (!qfmt::pair_schedule_fits(tiles, chunks_per_tile)) return QFMT_ERR_BAD_ARG;
    const long long total = tiles * chunks_per_tile;
    const qfmt::PairPiece pc = qfmt::pair_piece((int)(total / qfmt::kPlanPairs), (int)(total % qfmt::kPlanPairs), chunks_per_tile,
                                                chunks_per_tile * qfmt::kChunkKB, qfmt::kPlanPairs, pair, j);
    out[0] = pc.tile; out[1] = pc.kb_begin / qfmt::kChunkKB; out[2] = pc.num_kb / qfmt::kChunkKB; out[3] = pc.partial; out[4] = pc.head;
    const long long range = (total + qfmt::kPlanPairs - 1) / qfmt::kPlanPairs;
    out[5] = (int32_t)((range + chunks_per_tile - 1) / chunks_per_tile + 1);
    return QFMT_OK;
}

extern "C" int qfmt_gemm_tile_policy(int policy) {
    if (policy < 0 || policy > 3) return QFMT_ERR_BAD_ARG;
    qfmt::g_tile_policy.store(policy);
    return QFMT_OK;
}

extern "C" size_t qfmt_gemm_workspace_bytes(const qfmt_matrix_t* A, const qfmt_matrix_t* B) {
    if (A == nullptr || B == nullptr || A->rows < 0 || A->cols < 0 || B->rows < 0 || B->cols < 0)
        return qfmt::kWorkspaceHeader;
    const int64_t M = A->trans ? A->cols : A->rows, K = A->trans ? A->rows : A->cols;
    const int64_t N = B->trans ? B->rows : B->cols;
    if (M <= 0 || N <= 0 || K <= 0 || M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return qfmt::kWorkspaceHeader;
    const qfmt::DensePlan plan = qfmt::plan_dense(M, N, K);
    if (plan.sk) return qfmt::kWorkspaceHeader + qfmt::kSkFlagBytes;
    return qfmt::kWorkspaceHeader + (plan.splits > 1 ? (size_t)plan.splits * (size_t)M * (size_t)N * sizeof(float) : 0);
}

extern "C" size_t qfmt_gemm_packed16_workspace_bytes(const qfmt_matrix16_t* A, const qfmt_matrix16_t* B) {
    if (A == nullptr || B == nullptr || A->rows < 0 || A->cols < 0 || B->rows < 0 || B->cols < 0)
        return qfmt::kWorkspaceHeader;
    const int64_t M = A->trans ? A->cols : A->rows, K = A->trans ? A->rows : A->cols;
    const int64_t N = B->trans ? B->rows : B->cols;
    if (M <= 0 || N <= 0 || K <= 0 || M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return qfmt::kWorkspaceHeader;
    const qfmt::DensePlan plan = qfmt::plan_dense(M, N, (K + 1) / 2, 2);
    if (plan.sk) return qfmt::kWorkspaceHeader + qfmt::kSkFlagBytes;
    return qfmt::kWorkspaceHeader + (plan.splits > 1 ? (size_t)plan.splits * (size_t)M * (size_t)N * sizeof(float) : 0);
}

extern "C" int qfmt_device_status(void* d_workspace, void* stream) {
    if (d_workspace == nullptr) return QFMT_ERR_BAD_ARG;
    if (reinterpret_cast<uintptr_t>(d_workspace) & 7u) return QFMT_ERR_BAD_ARG;
    unsigned long long words[2] = {0, 0};
    QFMT_CUDA_TRY(cudaMemcpyAsync(words, d_workspace, sizeof(words), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    QFMT_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    // an error counts only if it carries the tag of the launch that last used the area (GemmParams::status)
    if (words[1] != 0 && (words[0] >> 16) == words[1]) return -(int)(words[0] & 0xFFFFu);
    return QFMT_OK;
}


extern "C" int qfmt_selftest_bounded_wait(void* d_status, uint32_t limit_cycles, int32_t* d_trace, void* stream) {
    if (d_status == nullptr || d_trace == nullptr) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_status) & 7u) || (reinterpret_cast<uintptr_t>(d_trace) & 3u)) return QFMT_ERR_BAD_ARG;
    if (limit_cycles == 0 || limit_cycles > (1u << 24)) return QFMT_ERR_BAD_ARG;  // at most a few milliseconds
    qfmt::DeviceInfo dev;
    int rc = qfmt::current_device(&dev);
    if (rc != QFMT_OK) return rc;
    QFMT_CUDA_TRY(cudaMemsetAsync(d_trace, 0, 4 * sizeof(int32_t), (cudaStream_t)stream));
    qfmt::bounded_wait_selftest_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(
        reinterpret_cast<unsigned long long*>(d_status), qfmt::next_launch_tag(), limit_cycles, d_trace);
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}

// ------------------------------------------------------------------------------------------------
// Variant with built-in scratch memory (no counterpart in the paper; see include/qfmt.h).
// ------------------------------------------------------------------------------------------------
namespace qfmt {
namespace {

constexpr size_t kBuiltinScratchBytes = (size_t)16 << 20;  // 16 MiB per GPU that loads the library

// The status area's verdict as one int32 (what qfmt_device_status computes on the host).
__global__ void status_word_kernel(const unsigned long long* status, int32_t* out) {
    const unsigned long long w0 = status[0], w1 = status[1];
    *out = (w1 != 0 && (w0 >> 16) == w1) ? -(int32_t)(w0 & 0xFFFFu) : 0;
}

// Lives in every device's copy of the module.  In host code this name is only a handle for
// cudaGetSymbolAddress: it is not a device address and must never be handed to a kernel.
static __device__ __align__(256) unsigned char g_builtin_scratch[kBuiltinScratchBytes];

// Device address of g_builtin_scratch on the current device, looked up once per device.
int builtin_scratch_address(void** out) {
    constexpr int kMaxDevices = 64;
    static std::atomic<void*> cached[kMaxDevices];
    int dev = 0;
    QFMT_CUDA_TRY(cudaGetDevice(&dev));
    void* p = (dev >= 0 && dev < kMaxDevices) ? cached[dev].load() : nullptr;
    if (p == nullptr) {
        QFMT_CUDA_TRY(cudaGetSymbolAddress(&p, g_builtin_scratch));  // with `dev` current
        if (p == nullptr) { set_last_cuda_error((int)cudaErrorInvalidSymbol); return QFMT_ERR_CUDA; }
        if (dev >= 0 && dev < kMaxDevices) cached[dev].store(p);
    }
    *out = p;
    return QFMT_OK;
}

}  // namespace
}  // namespace qfmt

extern "C" int qfmt_gemm_builtin_scratch(const qfmt_matrix_t* A, const qfmt_matrix_t* B, float* d_C, int64_t ldc,
                                         const qfmt_format_t* fmt, int32_t* d_status_out, void* stream) {
    // Everything the host can check comes first, so that an error return has enqueued nothing.  The
    // checks use a stand-in workspace address; the array's real address is looked up afterwards.
    int64_t M = 0, N = 0, K = 0;
    alignas(16) static const char placeholder[16] = {};
    if (A == nullptr || B == nullptr) return QFMT_ERR_BAD_ARG;
    int rc = qfmt::validate_gemm_args(A, B, d_C, ldc, fmt, placeholder, qfmt::kBuiltinScratchBytes, &M, &N, &K);
    if (rc != QFMT_OK) return rc;
    if (reinterpret_cast<uintptr_t>(d_status_out) & 3u) return QFMT_ERR_BAD_ARG;
    if (qfmt_gemm_workspace_bytes(A, B) > qfmt::kBuiltinScratchBytes) return QFMT_ERR_SCRATCH_LIMIT;
    void* scratch = nullptr;
    rc = qfmt::builtin_scratch_address(&scratch);
    if (rc != QFMT_OK) return rc;
    // The array still holds what the previous call left.  A product with work to do names its launch in
    // the status area at the array's head, which makes older entries there void; the area is cleared
    // here only for the call that enqueues no kernel (M or N zero), which must not report an older
    // call's status.
    if (M == 0 || N == 0) QFMT_CUDA_TRY(cudaMemsetAsync(scratch, 0, 16, (cudaStream_t)stream));
    rc = qfmt::gemm_device(A, B, d_C, ldc, fmt, scratch, qfmt::kBuiltinScratchBytes, (cudaStream_t)stream);
    if (rc != QFMT_OK) return rc;
    if (d_status_out != nullptr) {
        qfmt::status_word_kernel<<<1, 1, 0, (cudaStream_t)stream>>>(reinterpret_cast<const unsigned long long*>(scratch),
                                                                    d_status_out);
        QFMT_CUDA_TRY(cudaGetLastError());
    }
    return QFMT_OK;
}
