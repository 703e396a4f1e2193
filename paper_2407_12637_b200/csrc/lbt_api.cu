// Status names (host only).
#include "lbt_common.cuh"

extern "C" const char* lbt_status_string(lbt_status status) {
    switch (status) {
        case LBT_OK: return "LBT_OK";
        case LBT_ERR_INVALID_ARG: return "LBT_ERR_INVALID_ARG";
        case LBT_ERR_ALIGNMENT: return "LBT_ERR_ALIGNMENT";
        case LBT_ERR_UNSUPPORTED_BITS: return "LBT_ERR_UNSUPPORTED_BITS";
        case LBT_ERR_ACC_RANGE: return "LBT_ERR_ACC_RANGE";
        case LBT_ERR_WORKSPACE: return "LBT_ERR_WORKSPACE";
        case LBT_ERR_CUDA: return "LBT_ERR_CUDA";
        case LBT_ERR_NONFINITE: return "LBT_ERR_NONFINITE";
        case LBT_ERR_TIMEOUT: return "LBT_ERR_TIMEOUT";
        case LBT_ERR_UNSUPPORTED: return "LBT_ERR_UNSUPPORTED";
        default: return "LBT_ERR_UNKNOWN";
    }
}
