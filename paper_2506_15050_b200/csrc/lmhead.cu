// LM-head variant of the fused policy loss (logits = hidden x weight on the tensor cores).
#include "common.cuh"

namespace tppo {
size_t lmhead_workspace_bytes(int64_t, int32_t, int32_t) { return kWsAlign; }
}  // namespace tppo

TPPO_API int tppo_lmhead_logprob_fwd_bwd(const void*, const void*, int64_t, int32_t, int32_t,
                                         const int32_t*, const int32_t*, const float*, const float*,
                                         int64_t, float, float, float, float*, float*, float*,
                                         int32_t*, void*, void*, void*, size_t, void*) {
    return TPPO_ERR_UNSUPPORTED;
}
