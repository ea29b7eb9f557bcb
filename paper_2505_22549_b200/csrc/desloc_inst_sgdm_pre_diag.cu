// desloc_step_kernel instantiations: SGDM, pre-average ordering, with norm diagnostics.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_sgdm_pre_diag(bool bf16, int mt, int mask) {
    return lookup_unit<OPT_SGDM, false, true>(bf16, mt, mask);
}
}  // namespace desloc
