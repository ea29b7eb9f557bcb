// desloc_step_kernel instantiations: ADOPT, pre-average ordering.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_adopt_pre(bool bf16, int mt, int mask) {
    if (mt == 1) return mask == 0 ? lookup_local<OPT_ADOPT>(bf16) : nullptr;
    return lookup_sync<OPT_ADOPT, false>(bf16, mt, mask);
}
}  // namespace desloc
