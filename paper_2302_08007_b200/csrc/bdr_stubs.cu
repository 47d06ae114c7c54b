// Entry points whose kernels are not built yet.
#include "bdr.h"
extern "C" {
int64_t bdr_qsnr_workspace_bytes(int) { return 0; }
int bdr_qsnr(const bdr_config_t*, int, const void*, bdr_dtype_t, int64_t, int64_t, int64_t, int, double*, void*, int64_t, void*) { return BDR_ERR_UNSUPPORTED; }
int mx_gemm(const bdr_config_t*, const bdr_planes_t*, const bdr_config_t*, const bdr_planes_t*, int64_t, int64_t, int64_t, float*, int64_t, void*) { return BDR_ERR_UNSUPPORTED; }
}
