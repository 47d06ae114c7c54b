// Entry points whose kernels are not built yet.
#include "bdr.h"
extern "C" {
int mx_gemm(const bdr_config_t*, const bdr_planes_t*, const bdr_config_t*, const bdr_planes_t*, int64_t, int64_t, int64_t, float*, int64_t, void*) { return BDR_ERR_UNSUPPORTED; }
}
