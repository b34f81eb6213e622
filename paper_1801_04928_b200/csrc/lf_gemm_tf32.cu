// TF32 tensor-core contraction for the mini-batch weight gradient (Eq. bp4 summed over samples).
#include "lf_internal.h"

bool lf_tf32_supported(const lf_ctx*) { return false; }
int lf_gw_gemm_tf32(lf_ctx*, const float*, const float*, float*, cudaStream_t, int*)
{
    return LF_EINVAL;
}
void lf_tf32_release(lf_ctx*) {}
