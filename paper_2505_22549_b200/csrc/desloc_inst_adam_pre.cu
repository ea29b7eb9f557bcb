// desloc_step_kernel instantiations: ADAM, pre-average ordering.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_adam_pre(bool bf16, int mt, int mask) {
    if (mt == 1) return mask == 0 ? lookup_local<OPT_ADAM>(bf16) : nullptr;
    return lookup_sync<OPT_ADAM, false>(bf16, mt, mask);
}
}  // namespace desloc
