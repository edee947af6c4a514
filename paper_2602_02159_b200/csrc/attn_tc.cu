// placeholder until the tensor-core kernels land
#include "focus_common.cuh"
bool attn_tc_supported(const focus_ctx*, const AttnArgs&) { return false; }
focus_status launch_attn_tc(focus_ctx*, const AttnArgs&, cudaStream_t) { return FOCUS_ERR_UNSUPPORTED; }
size_t attn_tc_workspace(const focus_shape*, int, int, int) { return 0; }
bool sink_tc_supported(const focus_ctx*, const focus_shape*, int) { return false; }
focus_status launch_sink_colsum_tc(focus_ctx*, const focus_shape*, const void*, int, const int32_t*, const int32_t*, int,
                                   const void*, const float*, float*, WsAlloc&, cudaStream_t) { return FOCUS_ERR_UNSUPPORTED; }
