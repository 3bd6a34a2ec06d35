// Placeholder: tensor-core path not wired yet.
#include "prefill_tc.h"
namespace griffin {
bool prefill_tc_supported(const griffin_ff_desc *, int) { return false; }
griffin_status launch_prefill_tc(const griffin_ff_desc *, const griffin_ff_weights *, const void *, int, void *,
                                 __nv_bfloat16 *, float *, float *, int *, void *, cudaStream_t) {
    return GRIFFIN_ERR_UNSUPPORTED;
}
}  // namespace griffin
