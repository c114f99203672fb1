// Dynamic loss scaling kept on the device (Section II: the loss is scaled so that small
// gradients stay representable; Section V trains "with DLS").  The paper cites the technique and
// states no rule; the one implemented is the common one: a step whose gradient tensors held any
// overflow, infinity or NaN is skipped and the scale is multiplied by `backoff`; after
// `growth_interval` consecutive clean steps the scale is multiplied by `growth`.
//
// The controller reads the statistics records the rounding pass wrote for the step's gradient
// tensors and updates a small state record in device memory; qfmt_quantize_stats_dls reads the
// scale from that record, so a training loop never has to bring a count back to the host.
#include <cuda_runtime.h>
#include <stdint.h>

#include "common.cuh"

namespace qfmt {

int quantize_stats_device(const float* d_in, float* d_out, size_t n, const qfmt_format_t* fmt,
                          qfmt_stats_t* d_stats, int accumulate, cudaStream_t stream, const float* d_scale);

namespace {

constexpr int kDlsThreads = 256;

__global__ void __launch_bounds__(kDlsThreads)
dls_update_kernel(qfmt_dls_t* __restrict__ state, const qfmt_stats_t* __restrict__ stats, long long n_records) {
    __shared__ unsigned long long partial[kDlsThreads / 32];
    unsigned long long bad = 0ull;
    for (long long r = threadIdx.x; r < n_records; r += kDlsThreads)
        bad += stats[r].n_overflow + stats[r].n_nan + stats[r].n_inf_in;
    for (int off = 16; off > 0; off >>= 1) bad += __shfl_down_sync(0xFFFFFFFFu, bad, off);
    if ((threadIdx.x & 31) == 0) partial[threadIdx.x >> 5] = bad;
    __syncthreads();
    if (threadIdx.x != 0) return;
    bad = 0ull;
    for (int w = 0; w < kDlsThreads / 32; ++w) bad += partial[w];
    qfmt_dls_t s = *state;
    s.n_steps += 1;
    if (bad != 0ull) {
        const float v = __fmul_rn(s.scale, s.backoff);
        s.scale = v < s.min_scale ? s.min_scale : v;
        s.clean_steps = 0;
        s.skip = 1;
        s.n_skipped += 1;
    } else {
        s.skip = 0;
        s.clean_steps += 1;
        if (s.clean_steps >= s.growth_interval) {
            const float v = __fmul_rn(s.scale, s.growth);
            s.scale = v > s.max_scale ? s.max_scale : v;
            s.clean_steps = 0;
        }
    }
    *state = s;
}

}  // namespace
}  // namespace qfmt

extern "C" int qfmt_dls_update(qfmt_dls_t* d_state, const qfmt_stats_t* d_stats, int64_t n_records, void* stream) {
    if (d_state == nullptr || n_records < 0 || (n_records > 0 && d_stats == nullptr)) return QFMT_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(d_state) & 7u) || (reinterpret_cast<uintptr_t>(d_stats) & 7u)) return QFMT_ERR_BAD_ARG;
    qfmt::DeviceInfo dev;
    int rc = qfmt::current_device(&dev);
    if (rc != QFMT_OK) return rc;
    qfmt::dls_update_kernel<<<1, qfmt::kDlsThreads, 0, (cudaStream_t)stream>>>(d_state, d_stats, (long long)n_records);
    QFMT_CUDA_TRY(cudaGetLastError());
    return QFMT_OK;
}

extern "C" int qfmt_quantize_stats_dls(const float* d_in, float* d_out, size_t n, const qfmt_format_t* fmt,
                                       const qfmt_dls_t* d_state, qfmt_stats_t* d_stats, int accumulate, void* stream) {
    if (d_state == nullptr || (reinterpret_cast<uintptr_t>(d_state) & 7u)) return QFMT_ERR_BAD_ARG;
    return qfmt::quantize_stats_device(d_in, d_out, n, fmt, d_stats, accumulate, (cudaStream_t)stream, &d_state->scale);
}
