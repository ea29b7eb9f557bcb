// desloc_step_kernel instantiations: SGDM, post-average ordering.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_sgdm_post(bool bf16, int mt, int mask) {

    return lookup_sync<OPT_SGDM, true>(bf16, mt, mask);
}
}  // namespace desloc
