// Status names and the measurement taps (host only).
#include "lbt_common.cuh"

namespace lbt {

static cudaEvent_t g_tap[LBT_TIME_CLASSES][2];

void timing_begin(int kernel_class, cudaStream_t stream) {
    if (g_tap[kernel_class][0] != nullptr) cudaEventRecord(g_tap[kernel_class][0], stream);
}

void timing_end(int kernel_class, cudaStream_t stream) {
    if (g_tap[kernel_class][1] != nullptr) cudaEventRecord(g_tap[kernel_class][1], stream);
}

bool timing_armed(int kernel_class) { return g_tap[kernel_class][0] != nullptr; }

}  // namespace lbt

extern "C" lbt_status lbt_set_timing_events(int kernel_class, void* ev_start, void* ev_stop) {
    if (kernel_class < 0 || kernel_class >= LBT_TIME_CLASSES) return LBT_ERR_INVALID_ARG;
    if ((ev_start == nullptr) != (ev_stop == nullptr)) return LBT_ERR_INVALID_ARG;
    lbt::g_tap[kernel_class][0] = static_cast<cudaEvent_t>(ev_start);
    lbt::g_tap[kernel_class][1] = static_cast<cudaEvent_t>(ev_stop);
    return LBT_OK;
}

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
        case LBT_ERR_SCRATCH_LIMIT: return "LBT_ERR_SCRATCH_LIMIT";
        case LBT_ERR_BITS_MISMATCH: return "LBT_ERR_BITS_MISMATCH";
        default: return "LBT_ERR_UNKNOWN";
    }
}
