// Row-direction kernels instantiated for bf16 tensors (same source as bdr_row.cu, which covers fp32;
// two translation units so the two sets of template instantiations compile in parallel).
#define BDR_ROW_DTYPE __nv_bfloat16
#include "bdr_row.cu"
