// desloc_step_kernel instantiations: SGDM, pre-average ordering.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_sgdm_pre(bool bf16, int mt, int mask) {
    return lookup_unit<OPT_SGDM, false, false>(bf16, mt, mask);
}
}  // namespace desloc
