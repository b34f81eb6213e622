// Persistent single-launch backward pass for B = 1 (leapfrog CTA groups and the fused tile pass).
#include "lf_internal.h"

size_t lf_sync_words_needed(const lf_ctx* c) { return 64; }
bool lf_persistent_supported(const lf_ctx*, int) { return false; }
int lf_auto_variant(const lf_ctx*) { return LF_VARIANT_STREAMS; }
int lf_backward_persistent(lf_ctx*, int, const float*, const float*, const float*, const float*,
                           float*, float*, float*)
{
    return LF_EINVAL;
}
void lf_persistent_release(lf_ctx*) {}
