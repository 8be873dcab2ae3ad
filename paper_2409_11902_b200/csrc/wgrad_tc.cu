// Tensor-core weight-gradient kernel (placeholder until the tcgen05 path lands).
#include "ac_common.h"

namespace ac {
bool tc_supported(const Dims&) { return false; }
void plan_tc(const Dims&, WgradPlan*) {}
ac_status launch_wgrad_tc(const Dims&, const WgradPlan&, const void*, const void*, float*, void*,
                          cudaStream_t) {
    return AC_ERR_UNSUPPORTED;
}
}  // namespace ac
