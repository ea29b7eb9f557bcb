// Instantiation tables for desloc_step_kernel.  Each optimizer x averaging order x (with or
// without norm diagnostics) is its own translation unit (they compile in parallel); this header
// builds the (MT, mask) -> kernel table for one of them.
#pragma once
#include <utility>

#include "desloc_kernels.cuh"

namespace desloc {

template <int OPT, bool POST, bool DIAG, typename GT, int MT, int MASK>
const void *kernel_ptr() {
    return reinterpret_cast<const void *>(&desloc_step_kernel<OPT, MASK, MT, GT, POST, DIAG>);
}

// Masks FIRST..LAST for every MT in 2..MAX_MT.  LAST = 7 for Adam / ADOPT, 3 for SGDM (no
// second state).  FIRST = 0 for the pre-average units (mask 0, the local step, is the same
// code for either ordering) and 1 for the post-average ones.
template <int OPT, bool POST, bool DIAG, typename GT, int FIRST, int NMASK, int... I>
const void *pick_sync(int mt, int mask, std::integer_sequence<int, I...>) {
    static const void *const tbl[] = {
        kernel_ptr<OPT, POST, DIAG, GT, 2 + I / NMASK, FIRST + I % NMASK>()...};
    if (mt < 2 || mt > MAX_MT || mask < FIRST || mask >= FIRST + NMASK) return nullptr;
    return tbl[(mt - 2) * NMASK + (mask - FIRST)];
}

template <int OPT, bool POST, bool DIAG>
const void *lookup_sync(bool bf16, int mt, int mask) {
    constexpr int FIRST = POST ? 1 : 0;
    constexpr int NMASK = ((OPT == OPT_SGDM) ? 3 : 7) + 1 - FIRST;
    using Seq = std::make_integer_sequence<int, (MAX_MT - 1) * NMASK>;
    return bf16 ? pick_sync<OPT, POST, DIAG, bf16_t, FIRST, NMASK>(mt, mask, Seq{})
                : pick_sync<OPT, POST, DIAG, float, FIRST, NMASK>(mt, mask, Seq{});
}

// One unit per (optimizer, ordering, diagnostics).  mt = 1 is the one-replica-per-tile kernel
// (a single worker, or the local steps of more than MAX_MT workers); it lives in the pre units.
template <int OPT, bool POST, bool DIAG>
const void *lookup_unit(bool bf16, int mt, int mask) {
    if (mt == 1) {
        if constexpr (!POST) {
            if (mask != 0) return nullptr;
            return bf16 ? kernel_ptr<OPT, false, DIAG, bf16_t, 1, 0>() : kernel_ptr<OPT, false, DIAG, float, 1, 0>();
        }
        return nullptr;
    }
    return lookup_sync<OPT, POST, DIAG>(bf16, mt, mask);
}

#define DESLOC_DECLARE_UNIT(name) const void *lookup_##name(bool bf16, int mt, int mask)
DESLOC_DECLARE_UNIT(adam_pre);
DESLOC_DECLARE_UNIT(adam_post);
DESLOC_DECLARE_UNIT(adopt_pre);
DESLOC_DECLARE_UNIT(adopt_post);
DESLOC_DECLARE_UNIT(sgdm_pre);
DESLOC_DECLARE_UNIT(sgdm_post);
DESLOC_DECLARE_UNIT(adam_pre_diag);
DESLOC_DECLARE_UNIT(adam_post_diag);
DESLOC_DECLARE_UNIT(adopt_pre_diag);
DESLOC_DECLARE_UNIT(adopt_post_diag);
DESLOC_DECLARE_UNIT(sgdm_pre_diag);
DESLOC_DECLARE_UNIT(sgdm_post_diag);
#undef DESLOC_DECLARE_UNIT

}  // namespace desloc
