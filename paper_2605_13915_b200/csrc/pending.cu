// Entry points whose kernels are not written yet: they validate nothing and report MSD_ERR_UNSUPPORTED.
#include "host_common.h"

extern "C" {

size_t msd_gemm_dequant_bf16_workspace_bytes(int64_t, int64_t, int64_t) { return 0; }
msd_status_t msd_gemm_dequant_bf16(const void*, const int8_t*, const float*, int64_t, int64_t, int64_t, void*, msd_out_t,
                                   void*, size_t, void*) { return MSD_ERR_UNSUPPORTED; }
}  // extern "C"
