// desloc_step_kernel instantiations: SGDM, post-average ordering, with norm diagnostics.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_sgdm_post_diag(bool bf16, int mt, int mask) {
    return lookup_unit<OPT_SGDM, true, true>(bf16, mt, mask);
}
}  // namespace desloc
