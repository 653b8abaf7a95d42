// tcgen05 / TMEM / TMA implicit-GEMM convolutions. (Placeholder translation unit: no shape is taken yet.)
#include "pt_internal.h"

bool pt_sm100_conv_supported(const pt_ctx *, const pt_conv_desc *, int) { return false; }
size_t pt_sm100_conv_workspace(const pt_ctx *, const pt_conv_desc *, int) { return 0; }
pt_status pt_sm100_conv(pt_ctx *, const pt_conv_desc *, int, const void *, const void *, void *, void *, size_t, cudaStream_t)
{
    return PT_ERR_UNSUPPORTED;
}
