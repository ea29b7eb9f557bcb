// desloc_step_kernel instantiations: SGDM, post-average ordering.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_sgdm_post(bool bf16, int mt, int mask) {
    return lookup_unit<OPT_SGDM, true, false>(bf16, mt, mask);
}
}  // namespace desloc
