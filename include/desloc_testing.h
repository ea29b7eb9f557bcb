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

/*
 * Whether the step kernels stage their tiles through shared memory: -1 = the library decides (the
 * default: a launch of at most two blocks per SM of single-tile chunks skips the staging, since
 * it has nothing to overlap), 0 = stage whenever alignment allows, 1 = never (every chunk is
 * updated straight from global memory).  Results do not depend on it.  DESLOC_E_RANGE for other
 * values.
 */
DESLOC_API int desloc_testing_set_staging(desloc_ctx *ctx, int32_t mode);

/*
 * How often a thread block polls for its tile's copies before it gives up (default: about four
 * million polls).  polls = 0 makes every block give up at once: the step then stores nothing,
 * the blocks still let their copies land before they leave, and every later step call returns
 * DESLOC_E_DEVICE_WAIT -- the way the tests exercise the bounded-wait path without hanging or
 * faulting anything.  A negative value restores the default and clears the recorded failure.
 */
DESLOC_API int desloc_testing_set_wait_limit(desloc_ctx *ctx, int32_t polls);

#ifdef __cplusplus
}
#endif
#endif /* DESLOC_TESTING_H_ */
