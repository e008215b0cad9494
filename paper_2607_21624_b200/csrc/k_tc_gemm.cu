#include "fbl_internal.h"
bool gemm_tc_supported(const fbl_plan*, const GemmArgs&) { return false; }
cudaError_t launch_gemm_tc(const fbl_plan*, const GemmArgs&, void*, size_t, int32_t*, cudaStream_t) { return cudaErrorNotSupported; }
