// Shared host-side helpers of the library's translation units (status plumbing, device checks).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

#include "qfmt.h"

namespace qfmt {

// Records a failing CUDA call's code for qfmt_last_cuda_error().
void set_last_cuda_error(int code);

// Properties of the current device that the launch heuristics need; cached per device ordinal.
struct DeviceInfo {
    int ordinal;
    int cc_major;
    int sm_count;
};
// Returns QFMT_OK and fills *info, or QFMT_ERR_CUDA / QFMT_ERR_UNSUPPORTED_ARCH.
int current_device(DeviceInfo* info);

// Checks the fields of a format descriptor (Section IV-A: e <= 8, m <= 23; RNE only).
int validate_format(const qfmt_format_t* fmt);

#define QFMT_CUDA_TRY(expr)                                  \
    do {                                                     \
        cudaError_t err__ = (expr);                          \
        if (err__ != cudaSuccess) {                          \
            ::qfmt::set_last_cuda_error((int)err__);         \
            (void)cudaGetLastError();                        \
            return QFMT_ERR_CUDA;                            \
        }                                                    \
    } while (0)

// Programmatic dependent launch, device side.  A kernel launched by launch_overlapping may be placed on SMs
// that the kernel before it in the stream has left while that kernel still runs; grid_dependency_wait
// returns once that kernel has completed and its writes are visible (at once in an ordinary launch).
// grid_launch_dependents lets the next such launch be placed as soon as every CTA of this grid has
// executed it or exited.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Launch with programmatic stream serialization: the grid may be placed on SMs that the kernel before it
// in the stream has left (once all of that kernel's CTAs have passed their grid_launch_dependents), so its
// prologue overlaps that kernel's tail.  Only for kernels that execute grid_dependency_wait before their
// first access to global memory (the GEMM kernels, the split-K reduction, the layer-output pass).  After anything else in the
// stream (a copy, a memset, a kernel without grid_launch_dependents) it is an ordinary launch.
template <typename... P, typename... A>
cudaError_t launch_overlapping(void (*kernel)(P...), unsigned grid, unsigned block, size_t smem, cudaStream_t stream,
                               A&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(block, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<A>(args)...);
}

// Zeroes a few words (the hand-over words of the balanced schedule, a statistics record).  A kernel rather than a memset so that the launches
// around it can overlap (launch_overlapping): it lets the product that follows be placed at once, then waits
// for the kernel before it (which may be a product still reading these words), then clears them; the product
// that follows waits for this kernel, and so for both.
static __global__ void __launch_bounds__(256) zero_words_kernel(int* words, int n) {
    grid_launch_dependents();
    grid_dependency_wait();
    for (int i = threadIdx.x; i < n; i += 256) words[i] = 0;
}

}  // namespace qfmt
