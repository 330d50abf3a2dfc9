// Error strings and other small host-only entry points.
#include "common.cuh"

extern "C" const char* free_strerror(int code) {
    switch (code) {
        case FREE_OK: return "ok";
        case FREE_ERR_ARG: return "invalid argument (null pointer, negative count or bad enum)";
        case FREE_ERR_SHAPE: return "inconsistent or out-of-range dimensions";
        case FREE_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case FREE_ERR_UNSUPPORTED: return "configuration not supported by the kernels";
        case FREE_ERR_SIGMA: return "variance not positive and finite";
        case FREE_ERR_WORKSPACE: return "workspace missing or too small";
        case FREE_ERR_CUDA: return "CUDA call failed";
        case FREE_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        default: return "unknown error code";
    }
}
