// Entry points that do not belong to one kernel file: status strings, version.
#include "efq_common.cuh"

extern "C" const char* efq_status_string(efq_status_t status)
{
    switch (status) {
        case EFQ_OK: return "ok";
        case EFQ_ERR_INVALID_ARG: return "invalid argument";
        case EFQ_ERR_UNSUPPORTED: return "unsupported shape or variant";
        case EFQ_ERR_ALIGNMENT: return "pointer or leading dimension not aligned";
        case EFQ_ERR_WORKSPACE: return "workspace missing or too small";
        case EFQ_ERR_ARCH: return "device is not compute capability 10.x";
        case EFQ_ERR_CUDA: return "CUDA call failed";
        case EFQ_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case EFQ_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of the no-allocation entry point";
    }
    return "unknown status";
}

extern "C" const char* efq_version(void) { return "efq-b200 sm_100a " EFQ_FWD_KERNEL_REVISION; }

