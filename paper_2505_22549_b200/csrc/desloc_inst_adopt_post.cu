// desloc_step_kernel instantiations: ADOPT, post-average ordering.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_adopt_post(bool bf16, int mt, int mask) {
    return lookup_unit<OPT_ADOPT, true, false>(bf16, mt, mask);
}
}  // namespace desloc
