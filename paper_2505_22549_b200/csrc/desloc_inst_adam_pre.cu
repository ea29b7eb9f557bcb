// desloc_step_kernel instantiations: ADAM, pre-average ordering.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_adam_pre(bool bf16, int mt, int mask) {
    return lookup_unit<OPT_ADAM, false, false>(bf16, mt, mask);
}
}  // namespace desloc
