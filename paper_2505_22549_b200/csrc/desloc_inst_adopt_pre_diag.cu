// desloc_step_kernel instantiations: ADOPT, pre-average ordering, with norm diagnostics.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_adopt_pre_diag(bool bf16, int mt, int mask) {
    return lookup_unit<OPT_ADOPT, false, true>(bf16, mt, mask);
}
}  // namespace desloc
