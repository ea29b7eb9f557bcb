// desloc_step_kernel instantiations: ADAM, post-average ordering, with norm diagnostics.
#include "desloc_inst.cuh"

namespace desloc {
const void *lookup_adam_post_diag(bool bf16, int mt, int mask) {
    return lookup_unit<OPT_ADAM, true, true>(bf16, mt, mask);
}
}  // namespace desloc
