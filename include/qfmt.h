/*
 * qfmt — emulated 16-bit floating-point formats for mixed-precision training on one B200.
 *
 * C ABI of the hot path of "Representation range needs for 16-bit neural network training"
 * (arXiv 2103.15940): rounding fp32 tensors to a 1/e/m/{d,n} format while recording range
 * statistics, and contracting the rounded operands with wide accumulation.
 *
 * General rules
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  Every buffer is
 *     allocated, owned and freed by the caller; the library allocates no memory.
 *   - All GPU work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and the calls return without synchronising unless stated otherwise.
 *   - Every function returns a qfmt_status_t (0 = success, negative = error); nothing throws,
 *     prints or exits.  An error return means no GPU work was enqueued by that call.
 *   - The device must be of compute capability 10.x (built for sm_100a).
 */
#ifndef QFMT_H_
#define QFMT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    QFMT_OK = 0,
    QFMT_ERR_BAD_FORMAT = -1,  /* e, m, rounding or loss_scale outside the supported domain   */
    QFMT_ERR_BAD_ARG = -2,     /* NULL/misaligned pointer, bad dimension, workspace too small  */
    QFMT_ERR_UNSUPPORTED_ARCH = -3, /* current device is not compute capability 10.x           */
    QFMT_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed (see qfmt_last_cuda_error)  */
    QFMT_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired (reported via the status area) */
    QFMT_ERR_SCRATCH_LIMIT = -6 /* qfmt_gemm_builtin_scratch: the problem needs more than 16 MiB   */
} qfmt_status_t;

/*
 * A floating-point system s/e/p/d in the sense of Definition III.2 with s = 1:
 * e exponent bits, m explicitly stored mantissa bits (Table I's column "p"), and denormals
 * kept ("d") or flushed to zero ("n").  Bias is 2^(e-1)-1, so E_min = 1-bias, E_max = bias and
 * the smallest denormal is 2^(E_min-m) (Table I); the all-ones exponent field is inf/NaN.
 * Section IV-A fixes the domain of the rounding kernel: e <= 8, m <= 23.
 */
typedef struct {
    int32_t e;          /* exponent bits, 2..8                                               */
    int32_t m;          /* stored mantissa bits, 1..23 (qfmt_gemm requires m <= 10)          */
    int32_t denormals;  /* 1 = keep denormals ("d"), 0 = flush them to signed zero ("n")     */
    int32_t rounding;   /* 0 = round to nearest, ties to even; any other value is rejected   */
    float loss_scale;   /* finite and > 0; tensors are multiplied by it before rounding      */
} qfmt_format_t;

/*
 * Per-tensor range statistics (Section V: the fraction of denormal elements of every layer's
 * activations, weights and activation gradients is what the paper logs and tabulates).
 * hist[c] counts elements by the stored exponent field c of the ROUNDED value in the target
 * format: c = 0 zero or denormal, 1 .. 2^e-2 one bin per binade of normal numbers,
 * 2^e-1 inf or NaN; bins >= 2^e stay zero.
 *   n_total     elements seen
 *   n_zero_in   inputs that are +-0
 *   n_denormal  elements whose rounded value, before any flush, is a nonzero denormal of the
 *               format (with denormals flushed these are exactly the flushed elements)
 *   n_underflow finite nonzero inputs whose final result is +-0
 *   n_overflow  finite inputs whose final result is +-inf
 *   n_nan, n_inf_in  NaN / infinite inputs
 * The record lives in device memory.
 */
typedef struct {
    uint64_t hist[256];
    uint64_t n_total, n_zero_in, n_denormal, n_underflow, n_overflow, n_nan, n_inf_in, reserved;
} qfmt_stats_t;

/*
 * Round n fp32 elements to format *fmt (Section IV-A, the roundfp operation) after
 * multiplying each by fmt->loss_scale in IEEE single precision (Section II, loss scaling),
 * and record the range statistics of the result in the same pass.
 *
 *   d_in     device, n floats, 4-byte aligned (16-byte alignment of d_in and d_out, or equal
 *            misalignment of the two, selects the 128-bit path; otherwise a scalar path runs)
 *   d_out    device, n floats; receives the rounded values in fp32 containers (the low 23-m
 *            mantissa bits are zero).  May equal d_in (in place) or be NULL (statistics only).
 *            Partial overlap with d_in is an error the library cannot detect.
 *   fmt      host pointer, read during the call
 *   d_stats  device, 8-byte aligned, or NULL for no statistics
 *   accumulate  0: the record is cleared first; 1: counts are added to what it holds
 *
 * Overflow gives +-inf, NaN gives a quiet NaN with the input's sign, zeros and flushed or
 * underflowed results keep their sign.  n = 0 is valid (with accumulate = 0 it clears the
 * record).  The result is deterministic (integer counting only).
 * Errors: QFMT_ERR_BAD_FORMAT, QFMT_ERR_BAD_ARG, QFMT_ERR_UNSUPPORTED_ARCH, QFMT_ERR_CUDA.
 */
int qfmt_quantize_stats(const float* d_in, float* d_out, size_t n, const qfmt_format_t* fmt,
                        qfmt_stats_t* d_stats, int accumulate, void* stream);

/*
 * qfmt_quantize_stats with a batched transpose folded into the same pass: d_in is
 * [batch][rows][cols], d_out is [batch][cols][rows], both dense fp32; rounding, loss scale and
 * statistics exactly as above (the statistics do not depend on the element order).
 * This is how convolution operands reach the channels-last layouts qfmt_conv reads, without an
 * extra trip through memory: the rounding pass of Section IV-A touches every element anyway.
 *     activations NCHW -> NHWC:  batch = N, rows = C, cols = H*W
 *     filters     KCRS -> KRSC:  batch = K, rows = C, cols = R*S
 * d_out must not overlap d_in.  Each of batch, rows, cols < 2^31.
 */
int qfmt_quantize_stats_transpose(const float* d_in, float* d_out, int64_t batch, int64_t rows, int64_t cols,
                                  const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate,
                                  void* stream);

/*
 * 16-bit storage.  Section II: in mixed-precision training "activations and gradients are kept in
 * half-precision, halving the required storage and bandwidth".  qfmt_quantize_stats_pack16 is
 * qfmt_quantize_stats writing, instead of fp32 containers, the packed code of every rounded value:
 * sign | stored exponent field | mantissa in the low 1 + e + m bits of a 16-bit word (Definition
 * III.1 with Section III's special encodings: all-ones exponent = inf, or NaN with the top mantissa
 * bit set; all-zero exponent = zero / denormal).  For 1/5/10 and 1/8/7 these are the bits of IEEE
 * binary16 and of bfloat16.  6 bytes of traffic per element instead of 8.  qfmt_unpack16 expands
 * codes to the fp32 containers the contractions read.
 *   d_codes   device, n 16-bit words, 2-byte aligned (16-byte alignment of both pointers selects
 *             the 128-bit path)
 * Requires e + m <= 15 (QFMT_ERR_BAD_FORMAT otherwise).  Statistics, loss scale, accumulate, n = 0
 * and errors as for qfmt_quantize_stats.
 */
int qfmt_quantize_stats_pack16(const float* d_in, uint16_t* d_codes, size_t n, const qfmt_format_t* fmt,
                               qfmt_stats_t* d_stats, int accumulate, void* stream);
int qfmt_unpack16(const uint16_t* d_codes, float* d_out, size_t n, const qfmt_format_t* fmt, void* stream);

/*
 * Output of a layer as Section IV-A's worked example computes it, Y = R(R(acc) + R(B)): `acc` is
 * the matrix product of the layer (what qfmt_gemm or qfmt_conv wrote: rows x cols, row-major,
 * leading dimension ld_acc), `bias` has one entry per column.  Each acc element and each bias
 * entry is multiplied by fmt->loss_scale and rounded to the format exactly as
 * qfmt_quantize_stats does; the two rounded terms are added without error and the sum is rounded
 * once more.  One pass over memory instead of three (round, add, round).
 *
 *   d_acc    device, 4-byte aligned; rows x cols floats with leading dimension ld_acc >= cols
 *   d_bias   device, cols floats (the raw fp32 bias; it is rounded inside the call)
 *   d_out    device, rows x cols with leading dimension ld_out >= cols; may equal d_acc when
 *            ld_out == ld_acc (in place); other overlap is an error the library cannot detect.
 *            16-byte aligned pointers with cols, ld_acc, ld_out multiples of 4 select the
 *            128-bit path, anything else a scalar path.
 *   d_stats  device or NULL: statistics of the OUTPUT tensor Y, in which the exact sum
 *            R(acc) + R(B) plays the part the input plays in qfmt_quantize_stats: n_zero_in
 *            counts sums that are exactly zero, n_underflow nonzero sums that end as zero (only
 *            possible with denormals flushed), n_overflow finite sums that end as +-inf,
 *            n_inf_in / n_nan sums that are infinite / NaN (inf - inf included).
 *   accumulate  as in qfmt_quantize_stats
 * A zero sum is -0 only if both terms are -0; any NaN comes out as the positive quiet NaN.
 * Requires m <= 10 (QFMT_ERR_BAD_FORMAT otherwise): the sum is formed by one fp32 addition, which
 * for such formats is exact or harmless to the final rounding.  rows = 0 or cols = 0 is valid.
 * Errors: QFMT_ERR_BAD_FORMAT, QFMT_ERR_BAD_ARG, QFMT_ERR_UNSUPPORTED_ARCH, QFMT_ERR_CUDA.
 */
int qfmt_bias_quantize_stats(const float* d_acc, int64_t ld_acc, const float* d_bias, float* d_out, int64_t ld_out,
                             int64_t rows, int64_t cols, const qfmt_format_t* fmt, qfmt_stats_t* d_stats,
                             int accumulate, void* stream);

/*
 * The same layer-output pass with Y written as packed 16-bit codes (the encoding of
 * qfmt_quantize_stats_pack16) instead of fp32 containers, so that a layer whose operands are codes
 * (qfmt_gemm_packed16) hands codes to the next one: 6 bytes per element instead of 8, and no
 * separate packing pass.  Arguments as for qfmt_bias_quantize_stats except
 *   d_codes   device, 2-byte aligned; rows x cols codes with leading dimension ld_codes >= cols.
 *             8-byte aligned d_codes with 16-byte aligned d_acc and d_bias and cols, ld_acc,
 *             ld_codes multiples of 4 select the vector path, anything else a scalar path.
 * The codes are those of the containers qfmt_bias_quantize_stats would write (NaN: the positive
 * quiet NaN code).  Requires m <= 10 and e + m <= 15 (QFMT_ERR_BAD_FORMAT otherwise).
 * Errors: QFMT_ERR_BAD_FORMAT, QFMT_ERR_BAD_ARG, QFMT_ERR_UNSUPPORTED_ARCH, QFMT_ERR_CUDA.
 */
int qfmt_bias_quantize_stats_pack16(const float* d_acc, int64_t ld_acc, const float* d_bias, uint16_t* d_codes,
                                    int64_t ld_codes, int64_t rows, int64_t cols, const qfmt_format_t* fmt,
                                    qfmt_stats_t* d_stats, int accumulate, void* stream);

/*
 * Dynamic loss scaling with the scale kept in device memory.  Section II describes loss scaling
 * and Section V trains every format "with DLS" and without; the paper cites the technique and
 * states no rule, so the usual one is taken: a step whose gradient tensors held any overflow,
 * infinity or NaN is skipped and the scale is multiplied by `backoff` (not below min_scale);
 * after `growth_interval` consecutive clean steps it is multiplied by `growth` (not above
 * max_scale).  The record lives in DEVICE memory; the caller initialises it (scale, growth,
 * backoff, limits, growth_interval; the rest zero) and may read `skip` back, or pass the record
 * to its own update kernel, to leave out the weight update of a skipped step.
 */
typedef struct {
    float scale;              /* current loss scale                                              */
    float growth, backoff;    /* e.g. 2 and 0.5                                                  */
    float min_scale, max_scale;
    int32_t growth_interval;  /* clean steps before the scale grows, >= 1                        */
    int32_t clean_steps;      /* clean steps since the scale last changed                        */
    int32_t skip;             /* written by qfmt_dls_update: 1 = the step just checked is skipped */
    int32_t reserved;
    uint64_t n_steps, n_skipped;
} qfmt_dls_t;

/*
 * One controller step: sums n_overflow + n_nan + n_inf_in over the n_records consecutive
 * statistics records at d_stats (those of the step's gradient tensors, as written by the
 * rounding pass) and updates *d_state by the rule above.  Everything happens on `stream`; nothing
 * is copied to the host.  n_records = 0 counts as a clean step.
 * Errors: QFMT_ERR_BAD_ARG (NULL or misaligned pointer, negative count), QFMT_ERR_UNSUPPORTED_ARCH,
 * QFMT_ERR_CUDA.
 */
int qfmt_dls_update(qfmt_dls_t* d_state, const qfmt_stats_t* d_stats, int64_t n_records, void* stream);

/*
 * qfmt_quantize_stats with the loss scale read on the device from d_state->scale when the kernel
 * runs (fmt->loss_scale is ignored, though still validated).  A kernel enqueued after
 * qfmt_dls_update on the same stream sees the updated scale.
 */
int qfmt_quantize_stats_dls(const float* d_in, float* d_out, size_t n, const qfmt_format_t* fmt,
                            const qfmt_dls_t* d_state, qfmt_stats_t* d_stats, int accumulate, void* stream);

/*
 * The same operation on HOST buffers: copies h_in to the device, runs the kernel, copies the
 * rounded tensor (if h_out != NULL) and the statistics (if h_stats != NULL) back, and
 * SYNCHRONISES the stream before returning.  The caller lends device scratch:
 *   d_work   device, 16-byte aligned, at least qfmt_quantize_stats_host_work_bytes(n) bytes
 * For full copy speed h_in / h_out should be page-locked.  h_stats is overwritten.
 * Tensors of more than 2 Mi elements are moved in pieces on two internal streams (created once
 * per GPU, on first use), so that the copy to the device, the rounding and the copy back overlap;
 * the call still starts after the work already on `stream` and returns when everything is done.
 */
int qfmt_quantize_stats_host(const float* h_in, float* h_out, size_t n, const qfmt_format_t* fmt,
                             qfmt_stats_t* h_stats, void* d_work, size_t work_bytes, void* stream);
size_t qfmt_quantize_stats_host_work_bytes(size_t n);

/*
 * One GEMM operand: a row-major fp32 matrix in device memory whose elements already hold
 * values of the format (the output of qfmt_quantize_stats).  rows x cols is the STORED shape,
 * ld its leading dimension in elements; trans != 0 means the operand is the transpose of the
 * stored matrix, so the three products of a fully connected layer (Section V: forward,
 * activation gradient, weight gradient) need no copies:
 *     Y = X W        A = {X, trans 0},  B = {W, trans 0}
 *     dX = dY W^T    A = {dY, trans 0}, B = {W, trans 1}
 *     dW = X^T dY    A = {X, trans 1},  B = {dY, trans 0}
 * ptr must be 16-byte aligned and ld a multiple of 4 (the tiles are fetched by TMA).
 */
typedef struct {
    const float* ptr;
    int64_t rows, cols, ld;
    int32_t trans;
} qfmt_matrix_t;

/*
 * C = op(A) op(B) with exact products and fp32 accumulation: the FMACS instruction of
 * Section III-B, a32 = round(a32 + x16 * y16), which Section IV-A uses inside every matrix
 * multiply ("we do not round the products").  op(A) is M x K, op(B) is K x N, C is M x N
 * row-major with leading dimension ldc >= N (any 4-byte aligned d_C; 16-byte aligned rows
 * select vector stores).  Runs on the tcgen05 tensor cores as kind::tf32, which is exact for
 * operands of any format with e <= 8 and m <= 10; fmt states that format (m > 10 is rejected
 * with QFMT_ERR_BAD_FORMAT).  Operands are NOT re-rounded; feeding values with more than 10
 * mantissa bits loses the extra bits.  The accumulation order is fixed, so results are
 * reproducible run to run.  Against an exact sum the error of every element stays within
 * 2^-20 * sum_k |a_ik| |b_kj| whenever at least one operand carries mixed signs (every
 * workload the library is built for: signed weights or gradients meet the activations).
 * When BOTH operands are non-negative and heavy-tailed, the tensor core's truncation of each
 * 8-element partial sum goes one way and the error can exceed that bound, by less than a
 * factor of 2 (the tests pin both statements); no mode of this call restores the bound there.
 * fp32 denormal operands (only 1/8/m formats have them) are handled as the tensor core
 * handles them.
 *
 *   d_workspace  device, 16-byte aligned, at least 16 bytes; qfmt_gemm_workspace_bytes(A, B) is
 *                the size that lets the library run at full speed.  Holds a status area (first
 *                16 bytes: an error entry and the tag of the launch that last used the area; an
 *                entry counts only under that launch's tag, so the call clears nothing and the
 *                area's earlier contents never read as an error; read it with
 *                qfmt_device_status) and, for products with few output tiles and a
 *                long K, split-K partial sums (K is shared among CTAs and the parts are added
 *                in a fixed pairwise order).  A smaller workspace gets fewer or no splits: still
 *                correct and reproducible, but the last bits can differ from a run with the
 *                recommended size.  Calls that share a workspace must be ordered on one stream.
 * M = 0 or N = 0 is a no-op; K = 0 writes zeros.  Every device-side wait is bounded: if one
 * expires the kernel stops, the status area reports QFMT_ERR_TIMEOUT and C is undefined.
 * Errors: QFMT_ERR_BAD_FORMAT, QFMT_ERR_BAD_ARG (NULL or misaligned operand, ld too small,
 * mismatched K, workspace too small), QFMT_ERR_UNSUPPORTED_ARCH, QFMT_ERR_CUDA.
 */
int qfmt_gemm(const qfmt_matrix_t* A, const qfmt_matrix_t* B, float* d_C, int64_t ldc,
              const qfmt_format_t* fmt, void* d_workspace, size_t workspace_bytes, void* stream);
size_t qfmt_gemm_workspace_bytes(const qfmt_matrix_t* A, const qfmt_matrix_t* B);

/*
 * Forward pass of a fully connected layer as Section IV-A's worked example states it,
 *     Y = R( R( op(A) op(B) ) + R(bias) ),
 * with the FMACS contraction of qfmt_gemm inside and the statistics of Y recorded: qfmt_gemm
 * followed by qfmt_bias_quantize_stats, in one call and in place on d_Y.
 *
 * The library can also run both roundings, the bias addition and the counting inside the GEMM
 * kernel, on the sums while they are still in registers (contraction length K at most 1024 and
 * e <= 6), so that the fp32 product never goes to memory: see qfmt_linear_fusion_policy.  That
 * kernel sums K in one piece; its result has the bits of the two entry points called in turn
 * whenever qfmt_gemm does not split K for the problem (it may for products with few output tiles,
 * and then the two results agree within qfmt_gemm's error bound before the final roundings).
 *
 *   A, B, fmt        as for qfmt_gemm (operands hold format values); fmt->loss_scale must be 1
 *   d_bias           device, N floats (raw fp32; rounded inside the call)
 *   d_Y, ldy         device, M x N, leading dimension ldy >= N; receives Y (format values)
 *   d_stats, accumulate   as for qfmt_bias_quantize_stats (d_stats may be NULL)
 *   d_workspace      device, 16-byte aligned, at least qfmt_linear_forward_workspace_bytes(A, B)
 *                    bytes: status area as for qfmt_gemm (qfmt_device_status reads it), split-K
 *                    partial sums when the kernels run separately, and the rounded bias
 * Errors: as qfmt_gemm and qfmt_bias_quantize_stats; QFMT_ERR_BAD_FORMAT also for loss_scale != 1.
 */
int qfmt_linear_forward(const qfmt_matrix_t* A, const qfmt_matrix_t* B, const float* d_bias, float* d_Y, int64_t ldy,
                        const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate, void* d_workspace,
                        size_t workspace_bytes, void* stream);
size_t qfmt_linear_forward_workspace_bytes(const qfmt_matrix_t* A, const qfmt_matrix_t* B);

/*
 * Tuning and test control (no counterpart in the paper): how qfmt_linear_forward runs.
 *   0  automatic (default; currently two kernels, which measures faster: the epilogue's integer
 *      work in the GEMM kernel's few epilogue warps keeps the tensor cores waiting longer than
 *      the separate full-occupancy pass takes)
 *   1  epilogue inside the GEMM kernel whenever K <= 1024 and e <= 6
 *   2  always two kernels
 * Process-wide and not synchronised with calls in flight.  QFMT_ERR_BAD_ARG for other values.
 */
int qfmt_linear_fusion_policy(int policy);

/*
 * C = op(A) op(B) with FMAC-8 accumulation (Algorithm 1), for hardware that only offers the FMAC
 * instruction of Section III-B, a16 = round(a16 + x16 * y16) (one rounding, to the 16-bit format).
 * Every output is computed as the algorithm states: a format-precision accumulator takes eight
 * consecutive FMACs (k = 0..7, 8..15, ...), is added to a single-precision master accumulator
 * with an fp32 addition and restarts from zero; after the last (possibly shorter) group the master
 * accumulator is rounded to the format.  So, unlike qfmt_gemm, the result is fully specified:
 * C holds format values and is bit-exact against the definition.
 *
 *   A, B     as for qfmt_gemm (operands already hold values of the format; not re-rounded), but
 *            only 4-byte alignment is needed and any leading dimension >= the stored row length
 *   d_C      device, M x N floats, leading dimension ldc >= N, 4-byte aligned
 *   fmt      m <= 10 (QFMT_ERR_BAD_FORMAT otherwise); fmt->denormals selects whether the small
 *            accumulator and the result keep denormals or flush them; fmt->loss_scale is ignored
 *   d_stats  device or NULL: statistics of the OUTPUT tensor (Table II of the paper reports the
 *            denormal fraction of tensors produced this way), with the master accumulator in the
 *            role of the input of qfmt_quantize_stats; accumulate as there
 *   path     0 automatic; 1 the general kernel (integer/fp32 emulation of the FMAC on the ALUs);
 *            2 the native kernel (1/5/10 and 1/8/7 only, else QFMT_ERR_BAD_FORMAT), where the FMAC
 *            is the GPU's own binary16 / bfloat16 fused multiply-add.  Both give the same bits.
 * Plain-ALU work: no tensor-core instruction rounds its accumulator to 11 bits per product.
 * M = 0 or N = 0 is a no-op; K = 0 writes +0.  NaN results are the positive quiet NaN.
 * Errors: QFMT_ERR_BAD_FORMAT, QFMT_ERR_BAD_ARG, QFMT_ERR_UNSUPPORTED_ARCH, QFMT_ERR_CUDA.
 */
int qfmt_gemm_fmac8(const qfmt_matrix_t* A, const qfmt_matrix_t* B, float* d_C, int64_t ldc,
                    const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate, int path, void* stream);

/*
 * One operand of qfmt_gemm_packed16: a row-major matrix of packed 16-bit codes (the output of
 * qfmt_quantize_stats_pack16) in device memory; rows, cols, ld and trans as in qfmt_matrix_t.
 * ptr must be 16-byte aligned and ld a multiple of 8 (the tiles are fetched by TMA).
 */
typedef struct {
    const uint16_t* ptr;
    int64_t rows, cols, ld;
    int32_t trans;
} qfmt_matrix16_t;

/*
 * C = op(A) op(B) on operands stored as packed 16-bit codes, for the two formats whose codes are
 * words the tensor cores read directly: 1/5/10 (IEEE binary16) and 1/8/7 (bfloat16).  The same
 * FMACS contraction as qfmt_gemm (Section III-B: exact products, fp32 accumulation) with the same
 * operand conventions (the three products of a layer need no copies), run as tcgen05 kind::f16 at
 * twice the TF32 rate and with half the operand traffic; the summation is taken in the same three
 * levels with chunks of 128 K elements, and results stay within 2^-20 * sum_k |a_ik| |b_kj| of the
 * exact sum for the workloads this library targets.  Denormal codes are honoured; inf and NaN
 * codes propagate as in IEEE arithmetic.
 *
 *   d_C   device, M x N floats, leading dimension ldc >= N, 4-byte aligned
 *   fmt   {5, 10} or {8, 7}, QFMT_ERR_BAD_FORMAT otherwise (1/6/9 codes fit neither word: expand
 *         them with qfmt_unpack16 and use qfmt_gemm); denormals and loss_scale are ignored
 *   d_workspace, workspace_bytes   as for qfmt_gemm; qfmt_gemm_packed16_workspace_bytes(A, B) is
 *         the size that allows split K.  Status word and timeouts as for qfmt_gemm.
 * M = 0 or N = 0 is a no-op; K = 0 writes zeros.
 * Errors: QFMT_ERR_BAD_FORMAT, QFMT_ERR_BAD_ARG, QFMT_ERR_UNSUPPORTED_ARCH, QFMT_ERR_CUDA.
 */
int qfmt_gemm_packed16(const qfmt_matrix16_t* A, const qfmt_matrix16_t* B, float* d_C, int64_t ldc,
                       const qfmt_format_t* fmt, void* d_workspace, size_t workspace_bytes, void* stream);
size_t qfmt_gemm_packed16_workspace_bytes(const qfmt_matrix16_t* A, const qfmt_matrix16_t* B);

/*
 * Tuning and test control (no counterpart in the paper): which kernel dense products run on.
 *   0  automatic (default)
 *   1  single-CTA 128 x 256 tiles
 *   2  CTA-pair 256 x 256 tiles (tcgen05 cta_group::2; each SM stages half of the B operand)
 *   3  CTA-pair tiles under the balanced schedule wherever it applies (74 or more tiles, room for its
 *      flag words in the workspace): the tiles' K chunks are dealt among the 74 pairs in equal ranges,
 *      a tile cut by a range boundary is stored by one pair and completed by the next with an add at
 *      the destination, in a fixed order.  Never chosen automatically for dense products: measured
 *      slower than whole tiles on every product of the library's workloads.
 * Process-wide and not synchronised with calls in flight; results stay within the same bound under
 * every policy but their last bits may differ between policies.  Ask qfmt_gemm_workspace_bytes
 * again after changing it.  Returns QFMT_ERR_BAD_ARG for other values.
 */
int qfmt_gemm_tile_policy(int policy);
/*
 * The same for the forward and data-gradient products of qfmt_conv (filters larger than 1 x 1):
 *   0  automatic (default): CTA pairs, each CTA one M-tile of whole image rows and half of the filter
 *      columns, whenever there are two or more M-tiles
 *   1  always the single-CTA kernel
 *   2  CTA pairs on whole tiles
 *   3  CTA pairs under the balanced schedule wherever it applies
 * Ask qfmt_conv_workspace_bytes again after changing it.
 */
int qfmt_conv_tile_policy(int policy);

/*
 * Convolution layers (Section V: "matrix multiplications, at the core of fully connected and
 * convolution layers"): the three products of a unit-stride, zero-padded 2-D convolution,
 * computed as implicit GEMMs with the FMACS semantics of qfmt_gemm (exact products, fp32
 * accumulation, same error bound).  Nothing is unfolded in memory: tiles of the activation tensor
 * are fetched by TMA at each filter tap's offset and the padding is the copy engine's zero fill.
 *
 * All tensors are dense, channels-last, 16-byte aligned, and already hold format values (produce
 * them with qfmt_quantize_stats_transpose from NCHW / KCRS data, or qfmt_quantize_stats if they
 * are channels-last already):
 *     X  [n][h][w][c_in]      activations           Y, dY [n][oh][ow][c_out]
 *     W  [c_out][r][s][c_in]  filters               oh = h + 2 pad_h - r + 1, ow likewise
 *   op = QFMT_CONV_FWD    d_p = X,  d_q = W   d_out = Y   Y[n,oh,ow,co] = sum X[n,oh+r-pad_h,ow+s-pad_w,ci] W[co,r,s,ci]
 *   op = QFMT_CONV_DGRAD  d_p = dY, d_q = W   d_out = dX  dX[n,h,w,ci] = sum dY[n,h-r+pad_h,w-s+pad_w,co] W[co,r,s,ci]
 *   op = QFMT_CONV_WGRAD  d_p = dY, d_q = X   d_out = dW  dW[co,r,s,ci] = sum dY[n,oh,ow,co] X[n,oh+r-pad_h,ow+s-pad_w,ci]
 * Limits: c_in and c_out multiples of 32; output row length (ow; w for the data gradient) at
 * most 128 for the forward pass and the data gradient (none for the filter gradient, which takes
 * rows longer than 32 pixels in 32-pixel pieces); every tensor below 2^30 elements per
 * dimension product used as a GEMM extent.  Violations return QFMT_ERR_BAD_ARG.
 *   d_workspace  device, 16-byte aligned, >= qfmt_conv_workspace_bytes(op, geom) bytes: status
 *                area, and for the filter gradient the split-K partial sums (the long pixel
 *                dimension is split over CTAs and the parts are added in a fixed pairwise order,
 *                so results are reproducible).
 * Errors and the bounded-wait status area: as qfmt_gemm.
 */
typedef struct {
    int32_t n, c_in, h, w, c_out, r, s, pad_h, pad_w;
} qfmt_conv_t;
enum { QFMT_CONV_FWD = 0, QFMT_CONV_DGRAD = 1, QFMT_CONV_WGRAD = 2 };
int qfmt_conv(int32_t op, const qfmt_conv_t* geom, const float* d_p, const float* d_q, float* d_out,
              const qfmt_format_t* fmt, void* d_workspace, size_t workspace_bytes, void* stream);
size_t qfmt_conv_workspace_bytes(int32_t op, const qfmt_conv_t* geom);  /* 0 if geom is unsupported */

/*
 * The three products of a convolution layer with FMAC-8 accumulation (Section IV-A: FMAC-8 means
 * Algorithm 1 "or a matrix multiplication or convolution" whose sums are accumulated in its manner;
 * Table II's convolutional networks are trained this way).  Same tensors, layouts and operand order as
 * qfmt_conv (channels-last; unit stride, zero padding), same accumulation and output rules as
 * qfmt_gemm_fmac8: runs of eight FMACs in the 16-bit format, every run's sum added in fp32 to a
 * single-precision total, the total rounded to the format at the end; d_out holds format values and
 * is bit-exact against that definition.
 * The paper does not fix the order in which a convolution's reduction index is walked.  This library
 * walks it as the unfolded channels-last operand matrix would be:
 *     forward          filter taps row by row (r, then s), within a tap the input channels
 *     data gradient    filter taps row by row (r, then s), within a tap the output channels
 *     filter gradient  images, within an image the output rows, within a row the output pixels
 * A term whose input position lies in the zero padding is a term with a zero factor: it keeps its place
 * in its run of eight.
 *   geom     any positive sizes (no multiple-of-32 rule here); every tensor below 2^31 elements
 *   d_p, d_q, d_out   as for qfmt_conv, 4-byte aligned; operands hold values of the format
 *   fmt, d_stats, accumulate, path   as for qfmt_gemm_fmac8 (statistics of the output tensor)
 * Plain-ALU work, like qfmt_gemm_fmac8; the activation-like operand is gathered at the taps' offsets
 * while it is staged, nothing is unfolded in memory.
 * Errors: QFMT_ERR_BAD_FORMAT, QFMT_ERR_BAD_ARG, QFMT_ERR_UNSUPPORTED_ARCH, QFMT_ERR_CUDA.
 */
int qfmt_conv_fmac8(int32_t op, const qfmt_conv_t* geom, const float* d_p, const float* d_q, float* d_out,
                    const qfmt_format_t* fmt, qfmt_stats_t* d_stats, int accumulate, int path, void* stream);

/*
 * qfmt_gemm for callers that cannot allocate device memory.  (The paper has no counterpart of
 * this call; it exists for the way the library gets embedded.)
 *
 * qfmt_gemm needs a workspace that the caller allocates.  Some callers have no way to do that at
 * the point where they need the product: code that runs inside another framework's memory plan
 * and is handed only its input and output buffers; a real-time or safety-certified loop that is
 * forbidden to allocate once it has started; a process whose device memory has been given out
 * completely to a pool it does not own.  For them this variant keeps the workspace inside the
 * library: a fixed 16 MiB array that is part of the loaded GPU module, so every GPU that loads
 * libqfmt holds those 16 MiB from the first use of the library on that GPU until the process
 * ends.  The call itself performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *
 * Arguments A, B, d_C, ldc, fmt, stream: exactly as for qfmt_gemm, same results bit for bit.
 *   d_status_out  device, 4-byte aligned, or NULL.  If given, the product's status (QFMT_OK or
 *                 QFMT_ERR_TIMEOUT, one int32: what qfmt_device_status would report for a
 *                 caller-owned workspace) is written there on `stream` after the product; read it
 *                 with a copy of your own.
 * Limits and rules
 *   - A problem for which qfmt_gemm_workspace_bytes(A, B) exceeds 16 MiB (16 777 216 bytes) is
 *     refused with QFMT_ERR_SCRATCH_LIMIT and nothing is enqueued; use qfmt_gemm with your own
 *     workspace.  That figure counts the whole workspace: the 256-byte header that holds the
 *     status area as well as the partial sums of a product whose K dimension is split, so a
 *     product whose partial sums take exactly 16 MiB (1024 x 1024 outputs in four splits, say) is
 *     refused by those 256 bytes.  All argument checks of qfmt_gemm run before anything is
 *     enqueued, so every error return of this call leaves the stream untouched.
 *   - The first call on each GPU looks up the array's device address (a query, not an
 *     allocation).  Make that first call during set-up, before any stream capture begins.
 *   - All calls on one GPU share the one array and it keeps whatever the previous call left.
 *     The library clears what has to start at zero, but two calls whose GPU work can overlap
 *     (different streams without an ordering between them, or several host threads) race on it:
 *     keep every call on a GPU on one stream, or order them with events.
 * Errors: as qfmt_gemm, plus QFMT_ERR_SCRATCH_LIMIT.
 */
int qfmt_gemm_builtin_scratch(const qfmt_matrix_t* A, const qfmt_matrix_t* B, float* d_C, int64_t ldc,
                              const qfmt_format_t* fmt, int32_t* d_status_out, void* stream);

/*
 * Self-test of the error path the contraction kernels take when a device-side wait does not end
 * (every wait in them is bounded; see QFMT_ERR_TIMEOUT).  Launches one small block that waits, with
 * the same primitives, on a barrier nothing ever arrives on; the wait gives up after
 * `limit_cycles` SM cycles (1 .. 2^24, i.e. at most a few milliseconds), the block records
 * QFMT_ERR_TIMEOUT in the status area exactly as a contraction kernel would, its other warp notices
 * the block-wide abort flag, and the kernel returns normally: the context stays usable.
 *   d_status  device, 8-byte aligned, 16 bytes: a status area as at the head of a workspace (any
 *             contents); afterwards qfmt_device_status(d_status, stream) returns QFMT_ERR_TIMEOUT
 *   d_trace   device, four int32: [0] = 1 the waiting warp saw its wait expire, [1] = 1 the other warp
 *             left because of the abort flag, [2] = cycles waited, [3] unused
 * The paper has no counterpart; this is a diagnostic of the library.
 */
int qfmt_selftest_bounded_wait(void* d_status, uint32_t limit_cycles, int32_t* d_trace, void* stream);

/*
 * Host-only view of the balanced schedule of the CTA-pair kernels (tile policy 3, and the forward /
 * data-gradient products of qfmt_conv when their plan picks it): piece `j`, in the order pair `pair`
 * (0 .. 73) runs its pieces, of a product of `tiles` 256 x 256 tiles (>= 74) with `chunks_per_tile`
 * 64-element K chunks each.  Touches no device.
 *   out[0] tile index   out[1] first chunk within the tile   out[2] chunks (0: the pair has no piece j)
 *   out[3] 1 = the piece begins inside its tile and is added to what the pair before stored
 *   out[4] 1 = the piece ends before its tile does: the next pair finishes the tile
 *   out[5] the number of pieces the kernel provides for per pair
 * Returns QFMT_ERR_BAD_ARG for arguments outside these ranges or a product the schedule does not take.
 * The paper has no counterpart; this is a diagnostic of the library.
 */
int qfmt_selftest_pair_schedule(int64_t tiles, int32_t chunks_per_tile, int32_t pair, int32_t j, int32_t* out);

/*
 * Synchronises `stream` and returns what the status area at the head of a workspace (8-byte
 * aligned, 16 bytes) says about the launch that last used it: QFMT_OK, or the error that launch
 * recorded (QFMT_ERR_TIMEOUT), or QFMT_ERR_CUDA if the copy itself failed.  An area no launch has
 * used yet, whatever it holds, reads as QFMT_OK unless its two words happen to agree (2^-48).
 */
int qfmt_device_status(void* d_workspace, void* stream);

/* Last CUDA error code (cudaError_t as int) seen by a call that returned QFMT_ERR_CUDA. */
int qfmt_last_cuda_error(void);
/* Static, NUL-terminated description of a status code. */
const char* qfmt_status_string(int status);
/* Library version: major * 10000 + minor * 100 + patch. */
int qfmt_version(void);

#ifdef __cplusplus
}
#endif
#endif /* QFMT_H_ */
