// desloc_step_kernel instantiations: ADOPT, pre-average ordering.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_adopt_pre(bool bf16, int mt, int mask) {
    return lookup_unit<OPT_ADOPT, false, false>(bf16, mt, mask);
}
}  // namespace desloc
