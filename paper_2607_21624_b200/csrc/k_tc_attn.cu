#include "fbl_internal.h"
bool attn_fwd_tc_supported(const fbl_plan*) { return false; }
bool attn_bwd_tc_supported(const fbl_plan*) { return false; }
cudaError_t launch_attn_fwd_tc(const fbl_plan*, const void*, const void*, const void*, void*, float*, int32_t*, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t launch_attn_bwd_tc(const fbl_plan*, const void*, const void*, const void*, const void*, const void*, const float*, float*, float*, void*, void*, void*, int32_t*, cudaStream_t) { return cudaErrorNotSupported; }
