// Shared host-side helpers of the library's translation units (status plumbing, device checks).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

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

}  // namespace qfmt
