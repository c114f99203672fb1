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
// Every mbarrier wait is bounded; on expiry the thread records QFMT_ERR_TIMEOUT in the status
// word, raises a CTA-wide abort flag and every role drains to the common exit, where TMEM is
// released.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "common.cuh"
#include "ptx.cuh"

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
constexpr uint32_t kSmemBytes = kStages * kStageBytes + kOutBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr uint32_t kWaitLimit = 1u << 22;  // polls (with backoff) before a wait is declared dead

struct GemmParams {
    int M, N, K;
    long long ldc;
    float* C;
    int* status;
    int a_mn_major;  // op(A) stored with M contiguous
    int b_mn_major;  // op(B) stored with N contiguous
    int tiles_m, tiles_n;
    int tma_store;   // C base, row pitch and row length are multiples of 16 bytes: C is written by TMA
};

// Shared-memory matrix descriptor.  Addresses and offsets are stored in 16-byte units.
//   K-major tile (layout 2, 128-byte swizzle of 16-byte chunks): rows of 128 bytes (32 K
//       elements), 8-row groups 1024 bytes apart (stride offset); leading offset unused.
//   MN-major tile (layout 1, 128-byte swizzle of 32-byte chunks: the one layout 32-bit
//       operands may use when M/N is the contiguous dimension): blocks of [32 K-rows][128
//       bytes = 32 M/N elements]; leading offset = distance between blocks, stride offset =
//       distance between groups of 4 K-rows (512 bytes).
constexpr uint32_t kLayoutSw128 = 2, kLayoutSw128Base32 = 1;
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes,
                                              uint32_t layout) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version for sm_100
    d |= (uint64_t)layout << 61;
    return d;
}

__device__ __forceinline__ uint32_t make_idesc(int a_mn, int b_mn) {
    return (1u << 4)                     // D format: fp32
           | (2u << 7) | (2u << 10)      // A, B format: TF32
           | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16)
           | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

__device__ __forceinline__ void raise_timeout(const GemmParams& p, volatile int* abort_flag) {
    *abort_flag = 1;
    atomicCAS(p.status, 0, (int)QFMT_ERR_TIMEOUT);
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_tf32_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_c, const GemmParams p) {
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

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

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
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&tmap_a);
        ptx::prefetch_tensormap(&tmap_b);
        if (p.tma_store) ptx::prefetch_tensormap(&tmap_c);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const int num_tiles = p.tiles_m * p.tiles_n;
    const int num_kb = (p.K + kBK - 1) / kBK;

    // Registers are allocated per group of four warps: the producer/MMA group keeps 64 per thread,
    // the accumulate groups take 224 (128 running sums + 32 freshly loaded values + addressing).
    if (warp < 4) {
    ptx::setmaxnreg_dec<80>();
    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            for (int t = blockIdx.x; t < num_tiles && !*abort_flag; t += gridDim.x) {
                const int m0 = (t % p.tiles_m) * kBM;
                const int n0 = (t / p.tiles_m) * kBN;
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!ptx::mbar_wait_bounded(empty_bar(stage), phase ^ 1u, kWaitLimit)) {
                        raise_timeout(p, abort_flag);
                        break;
                    }
                    if (*abort_flag) break;
                    const uint32_t sa = tiles + stage * kStageBytes;
                    const uint32_t sb = sa + kABytes;
                    const int k0 = kb * kBK;
                    ptx::mbar_expect_tx(full_bar(stage), kStageBytes);
                    if (p.a_mn_major) {
                        for (int c = 0; c < kBM / 32; ++c)
                            ptx::tma_load_2d(sa + c * 4096u, &tmap_a, full_bar(stage), m0 + c * 32, k0);
                    } else {
                        ptx::tma_load_2d(sa, &tmap_a, full_bar(stage), k0, m0);
                    }
                    if (p.b_mn_major) {
                        for (int c = 0; c < kBN / 32; ++c)
                            ptx::tma_load_2d(sb + c * 4096u, &tmap_b, full_bar(stage), n0 + c * 32, k0);
                    } else {
                        ptx::tma_load_2d(sb, &tmap_b, full_bar(stage), k0, n0);
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            const uint32_t idesc = make_idesc(p.a_mn_major, p.b_mn_major);
            // per-MMA advance of the descriptor start address, in bytes
            const uint32_t a_step = p.a_mn_major ? 1024u : (uint32_t)kMmaK * 4u;
            const uint32_t b_step = p.b_mn_major ? 1024u : (uint32_t)kMmaK * 4u;
            const uint32_t a_lbo = p.a_mn_major ? 4096u : 16u, a_sbo = p.a_mn_major ? 512u : 1024u;
            const uint32_t b_lbo = p.b_mn_major ? 4096u : 16u, b_sbo = p.b_mn_major ? 512u : 1024u;
            const uint32_t a_lay = p.a_mn_major ? kLayoutSw128Base32 : kLayoutSw128;
            const uint32_t b_lay = p.b_mn_major ? kLayoutSw128Base32 : kLayoutSw128;
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_iter = 0;  // chunks issued so far: buffer = acc_iter & 1, phase = (acc_iter >> 1) & 1
            bool dead = false;
            for (int t = blockIdx.x; t < num_tiles && !dead; t += gridDim.x) {
                for (int kb0 = 0; kb0 < num_kb && !dead; kb0 += kChunkKB) {
                    const uint32_t acc = acc_iter & 1u, acc_phase = (acc_iter >> 1) & 1u;
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
                        if (*abort_flag) { dead = true; break; }
                        ptx::tc_fence_after_sync();
                        const uint32_t sa = tiles + stage * kStageBytes;
                        const uint32_t sb = sa + kABytes;
#pragma unroll
                        for (int k = 0; k < kBK / kMmaK; ++k) {
                            const uint64_t da = make_desc(sa + k * a_step, a_lbo, a_sbo, a_lay);
                            const uint64_t db = make_desc(sb + k * b_step, b_lbo, b_sbo, b_lay);
                            ptx::mma_tf32(d_tmem, da, db, idesc, (kb != kb0 || k != 0) ? 1u : 0u);
                        }
                        ptx::mma_commit(empty_bar(stage));  // stage reusable once these MMAs have read it
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                    if (dead) break;
                    ptx::mma_commit(acc_full_bar(acc));      // chunk sum complete
                    ++acc_iter;
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
        for (int t = blockIdx.x; t < num_tiles && !dead; t += gridDim.x) {
            const int m0 = (t % p.tiles_m) * kBM;
            const int n0 = (t / p.tiles_m) * kBN;
            float sum[128];  // level-1 running sums; 0 + x is exact, so a group's first chunk needs no special case
#pragma unroll
            for (int j = 0; j < 128; ++j) sum[j] = 0.0f;
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
                    for (int j = 0; j < 32; ++j) {
                        sum[pair * 64 + j] = __fadd_rn(sum[pair * 64 + j], __uint_as_float(ra[j]));
                        sum[pair * 64 + 32 + j] = __fadd_rn(sum[pair * 64 + 32 + j], __uint_as_float(rb[j]));
                    }
                }
                ++acc_iter;
                const bool last = kb0 + kChunkKB >= num_kb;
                if (!last && ++in_group < kFlushChunks) continue;
                // ---- move the level-1 sums to C (level 2): registers -> swizzled shared boxes -> TMA.
                // The first group of a tile is stored, later groups are added at the destination.
                if (p.tma_store && flushed) {
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
                        *reinterpret_cast<float4*>(box + lane * 32 + ((c ^ (lane & 7)) << 2)) =
                            make_float4(sum[j], sum[j + 1], sum[j + 2], sum[j + 3]);
                    }
                    if (p.tma_store) {
                        ptx::fence_proxy_async();
                        __syncwarp();
                        if (lane == 0) {
                            if (row0 < p.M && col0 < p.N) {
                                const uint32_t src = my_stage_addr + (pass & 1) * kOutBoxBytes;
                                if (flushed) ptx::tma_reduce_add_2d(&tmap_c, src, col0, row0);
                                else ptx::tma_store_2d(&tmap_c, src, col0, row0);
                            }
                            ptx::bulk_commit();  // committed even when empty: the wait above counts groups
                        }
                    } else {
                        __syncwarp();
                        for (int r = 0; r < 32; ++r) {
                            const int row = row0 + r;
                            if (row >= p.M) break;
                            const int c = lane;
                            if (col0 + c < p.N) {
                                float* g = p.C + (long long)row * p.ldc + col0 + c;
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
                    for (int j = 0; j < 128; ++j) sum[j] = 0.0f;
                }
            }
            if (dead) break;
        }
        if (lane == 0) ptx::bulk_wait_all();  // shared memory stays valid until the last copy has read it
        __syncwarp();
    }

    // ------------------------------ common exit ------------------------------
    ptx::tc_fence_before_sync();
    __syncthreads();
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

// 2-D fp32 tensor map with dim0 contiguous; box (box0, box1); zero fill out of bounds.
// Swizzle: 16-byte chunks within 128 bytes for K-major tiles and for C, 32-byte chunks for
// MN-major operand tiles.
int make_map_2d(CUtensorMap* map, const float* base, uint64_t dim0, uint64_t dim1, uint64_t ld_elems,
                uint32_t box0, uint32_t box1, bool mn_major) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (fn == nullptr) { set_last_cuda_error((int)cudaErrorSymbolNotFound); return QFMT_ERR_CUDA; }
    cuuint64_t dims[2] = {dim0, dim1};
    cuuint64_t strides[1] = {ld_elems * sizeof(float)};
    cuuint32_t box[2] = {box0, box1};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE,
                    mn_major ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_last_cuda_error(100000 + (int)r); return QFMT_ERR_CUDA; }
    return QFMT_OK;
}

}  // namespace

int gemm_device(const qfmt_matrix_t* A, const qfmt_matrix_t* B, float* d_C, int64_t ldc, const qfmt_format_t* fmt,
                void* d_workspace, size_t workspace_bytes, cudaStream_t stream) {
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
    if (M == 0 || N == 0) return QFMT_OK;
    if (A->ptr == nullptr && K != 0) return QFMT_ERR_BAD_ARG;
    if (B->ptr == nullptr && K != 0) return QFMT_ERR_BAD_ARG;
    if (d_C == nullptr || (reinterpret_cast<uintptr_t>(d_C) & 3u)) return QFMT_ERR_BAD_ARG;
    // TMA needs 16-byte aligned bases and row pitches
    if ((reinterpret_cast<uintptr_t>(A->ptr) & 15u) || (reinterpret_cast<uintptr_t>(B->ptr) & 15u) ||
        (A->ld & 3) || (B->ld & 3))
        return QFMT_ERR_BAD_ARG;
    DeviceInfo dev;
    rc = current_device(&dev);
    if (rc != QFMT_OK) return rc;

    int* status = reinterpret_cast<int*>(d_workspace);
    QFMT_CUDA_TRY(cudaMemsetAsync(status, 0, 16, stream));
    if (K == 0) {
        QFMT_CUDA_TRY(cudaMemset2DAsync(d_C, (size_t)ldc * sizeof(float), 0, (size_t)N * sizeof(float), (size_t)M, stream));
        return QFMT_OK;
    }

    GemmParams p;
    p.M = (int)M; p.N = (int)N; p.K = (int)K;
    p.ldc = ldc;
    p.C = d_C;
    p.status = status;
    p.a_mn_major = A->trans ? 1 : 0;
    p.b_mn_major = B->trans ? 0 : 1;
    p.tiles_m = (int)((M + kBM - 1) / kBM);
    p.tiles_n = (int)((N + kBN - 1) / kBN);
    // TMA stores clip at 16-byte granularity along the row, so N must be a multiple of 4 as well.
    p.tma_store = ((reinterpret_cast<uintptr_t>(d_C) & 15u) == 0 && (ldc & 3) == 0 && (N & 3) == 0) ? 1 : 0;

    CUtensorMap ma, mb, mc;
    if (p.a_mn_major) rc = make_map_2d(&ma, A->ptr, (uint64_t)M, (uint64_t)K, (uint64_t)A->ld, 32, kBK, true);
    else rc = make_map_2d(&ma, A->ptr, (uint64_t)K, (uint64_t)M, (uint64_t)A->ld, kBK, kBM, false);
    if (rc != QFMT_OK) return rc;
    if (p.b_mn_major) rc = make_map_2d(&mb, B->ptr, (uint64_t)N, (uint64_t)K, (uint64_t)B->ld, 32, kBK, true);
    else rc = make_map_2d(&mb, B->ptr, (uint64_t)K, (uint64_t)N, (uint64_t)B->ld, kBK, kBN, false);
    if (rc != QFMT_OK) return rc;

    if (p.tma_store) rc = make_map_2d(&mc, d_C, (uint64_t)N, (uint64_t)M, (uint64_t)ldc, 32, 32, false);
    else mc = ma;  // unused by the kernel
    if (rc != QFMT_OK) return rc;

    static bool attr_set[64] = {};
    if (dev.ordinal < 0 || dev.ordinal >= 64 || !attr_set[dev.ordinal]) {
        QFMT_CUDA_TRY(cudaFuncSetAttribute(gemm_tf32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
        if (dev.ordinal >= 0 && dev.ordinal < 64) attr_set[dev.ordinal] = true;
    }
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int grid = num_tiles < dev.sm_count ? num_tiles : dev.sm_count;
    gemm_tf32_kernel<<<grid, kThreads, kSmemBytes, stream>>>(ma, mb, mc, p);
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}

}  // namespace qfmt

extern "C" int qfmt_gemm(const qfmt_matrix_t* A, const qfmt_matrix_t* B, float* d_C, int64_t ldc,
                         const qfmt_format_t* fmt, void* d_workspace, size_t workspace_bytes, void* stream) {
    return qfmt::gemm_device(A, B, d_C, ldc, fmt, d_workspace, workspace_bytes, (cudaStream_t)stream);
}

extern "C" size_t qfmt_gemm_workspace_bytes(const qfmt_matrix_t* A, const qfmt_matrix_t* B) {
    (void)A; (void)B;
    return 256;
}

extern "C" int qfmt_device_status(void* d_workspace, void* stream) {
    if (d_workspace == nullptr) return QFMT_ERR_BAD_ARG;
    int st = 0;
    QFMT_CUDA_TRY(cudaMemcpyAsync(&st, d_workspace, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    QFMT_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return st;
}


// ------------------------------------------------------------------------------------------------
// Variant with built-in scratch memory (no counterpart in the paper; see include/qfmt.h).
// ------------------------------------------------------------------------------------------------
namespace qfmt {
namespace {

constexpr size_t kBuiltinScratchBytes = (size_t)16 << 20;  // 16 MiB per GPU that loads the library

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
    if (A == nullptr || B == nullptr) return QFMT_ERR_BAD_ARG;
    if (reinterpret_cast<uintptr_t>(d_status_out) & 3u) return QFMT_ERR_BAD_ARG;
    if (qfmt_gemm_workspace_bytes(A, B) > qfmt::kBuiltinScratchBytes) return QFMT_ERR_SCRATCH_LIMIT;
    void* scratch = nullptr;
    int rc = qfmt::builtin_scratch_address(&scratch);
    if (rc != QFMT_OK) return rc;
    // The array still holds what the previous call left.  Only the status word at its head has
    // to start at zero; clear it here as well so that a call that enqueues no kernel (M or N zero)
    // does not report an older call's status.
    QFMT_CUDA_TRY(cudaMemsetAsync(scratch, 0, 16, (cudaStream_t)stream));
    rc = qfmt::gemm_device(A, B, d_C, ldc, fmt, scratch, qfmt::kBuiltinScratchBytes, (cudaStream_t)stream);
    if (rc != QFMT_OK) return rc;
    if (d_status_out != nullptr)
        QFMT_CUDA_TRY(cudaMemcpyAsync(d_status_out, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice,
                                      (cudaStream_t)stream));
    return QFMT_OK;
}
