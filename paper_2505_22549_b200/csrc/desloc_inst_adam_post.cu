// desloc_step_kernel instantiations: ADAM, post-average ordering.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_adam_post(bool bf16, int mt, int mask) {
    return lookup_unit<OPT_ADAM, true, false>(bf16, mt, mask);
}
}  // namespace desloc
