/*
 * desloc_testing.h -- hooks for the library's own tests.  NOT part of the API: nothing here is
 * needed to use the library, and it may change without notice.
 */
#ifndef DESLOC_TESTING_H_
#define DESLOC_TESTING_H_

#include "desloc.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * Cap the grid of the step kernels of this context at max_blocks thread blocks (0 = no cap, the
 * default: one block per chunk).  With a cap the blocks stride over the chunks (the runtime-M
 * kernel for sync steps of more than eight workers ignores the cap).  Results do not
 * depend on it; the tests use it to run the striding path, which the default launch never takes
 * below 2^31 chunks.  DESLOC_E_RANGE for a negative value.
 */
DESLOC_API int desloc_testing_set_max_blocks(desloc_ctx *ctx, int64_t max_blocks);

#ifdef __cplusplus
}
#endif
#endif /* DESLOC_TESTING_H_ */
