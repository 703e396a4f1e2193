// placeholder until the tensor-core path lands
#include "lbt_common.cuh"
extern "C" size_t lbt_workspace_bytes(int, const void*) { return 0; }
extern "C" lbt_status lbt_qgemm_dgrad(const void*, const void*, const float*, const float*, float*, int32_t*, int64_t, int64_t, int64_t, int, int, int32_t*, void*, size_t, void*) { return LBT_ERR_UNSUPPORTED; }
extern "C" lbt_status lbt_qgemm_wgrad(const void*, const void*, const float*, const float*, float*, int32_t*, int64_t, int64_t, int64_t, int, int, int32_t*, void*, size_t, void*) { return LBT_ERR_UNSUPPORTED; }
extern "C" lbt_status lbt_qconv_dgrad_wgrad(const lbt_conv_desc*, const void*, const void*, const void*, const float*, const float*, const float*, float*, float*, int32_t*, int32_t*, int, int, int, int32_t*, void*, size_t, void*) { return LBT_ERR_UNSUPPORTED; }
extern "C" lbt_status lbt_qconv_backward(const lbt_conv_desc*, const float*, const void*, const void*, const float*, const float*, lbt_interval_state*, lbt_grad_stats_t*, void*, float*, float*, int32_t*, int32_t*, int, void*, size_t, void*) { return LBT_ERR_UNSUPPORTED; }
