// Entry points that launch nothing: version and status strings.
#include "common.cuh"

extern "C" int matq_version(void) { return 100; }

extern "C" const char* matq_status_string(int status) {
    switch (status) {
        case MATQ_OK: return "ok";
        case MATQ_ERR_INVALID_ARG: return "invalid argument";
        case MATQ_ERR_UNSUPPORTED: return "unsupported bit-width";
        case MATQ_ERR_SHAPE: return "unsupported shape";
        case MATQ_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case MATQ_ERR_WORKSPACE: return "workspace missing or too small";
        case MATQ_ERR_CUDA: return "CUDA runtime error";
        case MATQ_ERR_NONFINITE: return "non-finite weight";
        case MATQ_ERR_CAPACITY: return "overflow list capacity exceeded";
        case MATQ_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}
