// Status strings, version, device checks and format validation shared by the entry points.
#include <atomic>
#include <cmath>

#include "common.cuh"

namespace qfmt {

static std::atomic<int> g_last_cuda_error{0};

void set_last_cuda_error(int code) { g_last_cuda_error.store(code); }

int current_device(DeviceInfo* info) {
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cached_cc[kMaxDevices];
    static std::atomic<int> cached_sms[kMaxDevices];
    int dev = 0;
    QFMT_CUDA_TRY(cudaGetDevice(&dev));
    int cc = 0, sms = 0;
    if (dev >= 0 && dev < kMaxDevices && cached_cc[dev].load() != 0) {
        cc = cached_cc[dev].load();
        sms = cached_sms[dev].load();
    } else {
        QFMT_CUDA_TRY(cudaDeviceGetAttribute(&cc, cudaDevAttrComputeCapabilityMajor, dev));
        QFMT_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        if (dev >= 0 && dev < kMaxDevices) {
            cached_sms[dev].store(sms);
            cached_cc[dev].store(cc);
        }
    }
    info->ordinal = dev;
    info->cc_major = cc;
    info->sm_count = sms;
    return cc == 10 ? QFMT_OK : QFMT_ERR_UNSUPPORTED_ARCH;
}

int validate_format(const qfmt_format_t* fmt) {
    if (fmt == nullptr) return QFMT_ERR_BAD_ARG;
    if (fmt->e < 2 || fmt->e > 8) return QFMT_ERR_BAD_FORMAT;
    if (fmt->m < 1 || fmt->m > 23) return QFMT_ERR_BAD_FORMAT;
    if (fmt->denormals != 0 && fmt->denormals != 1) return QFMT_ERR_BAD_FORMAT;
    if (fmt->rounding != 0) return QFMT_ERR_BAD_FORMAT;
    if (!(fmt->loss_scale > 0.0f) || !std::isfinite(fmt->loss_scale)) return QFMT_ERR_BAD_FORMAT;
    return QFMT_OK;
}

}  // namespace qfmt

extern "C" int qfmt_last_cuda_error(void) { return qfmt::g_last_cuda_error.load(); }

extern "C" const char* qfmt_status_string(int status) {
    switch (status) {
        case QFMT_OK: return "ok";
        case QFMT_ERR_BAD_FORMAT: return "format descriptor outside the supported domain";
        case QFMT_ERR_BAD_ARG: return "bad argument";
        case QFMT_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x";
        case QFMT_ERR_CUDA: return "CUDA call failed";
        case QFMT_ERR_TIMEOUT: return "bounded device-side wait expired";
        case QFMT_ERR_SCRATCH_LIMIT: return "problem needs more scratch memory than the library's built-in 16 MiB";
        default: return "unknown status";
    }
}

extern "C" int qfmt_version(void) { return 100; }
