/* Plain C99 user of the DES-LOC C ABI: includes the public header as C, and calls the entry
 * points that need no GPU.  Exit code 0 = every check passed. */
#include <stdio.h>
#include <string.h>

#include "desloc.h"

static int fails = 0;
#define CHECK(c) do { if (!(c)) { printf("FAILED: %s (line %d)\n", #c, __LINE__); ++fails; } } while (0)

int main(void) {
    int64_t numel[3] = {10000, 5, 4096};
    desloc_config cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.M = 2;
    cfg.num_tensors = 3;
    cfg.numel = numel;
    cfg.opt = DESLOC_ADAM;
    cfg.grad_dtype = DESLOC_BF16;
    cfg.beta1 = 0.9f;
    cfg.beta2 = 0.999f;
    cfg.eps = 1e-8f;
    cfg.Kx = 4; cfg.Ku = 8; cfg.Kv = 16;

    CHECK(desloc_sync_mask(&cfg, 0) == (DESLOC_SYNC_X | DESLOC_SYNC_U | DESLOC_SYNC_V));
    CHECK(desloc_sync_mask(&cfg, 4) == DESLOC_SYNC_X);
    CHECK(desloc_sync_mask(&cfg, 8) == (DESLOC_SYNC_X | DESLOC_SYNC_U));
    CHECK(desloc_sync_mask(&cfg, 5) == 0);
    cfg.opt = DESLOC_SGDM;
    CHECK(desloc_sync_mask(&cfg, 16) == (DESLOC_SYNC_X | DESLOC_SYNC_U));
    cfg.opt = DESLOC_ADAM;

    CHECK(desloc_chunk_elems(&cfg) == 1024);   /* a small list: single-tile chunks (M = 2) */
    CHECK(desloc_chunk_elems(NULL) == DESLOC_E_NULL);
    int64_t out[3 * 8];
    int64_t n = desloc_plan_chunks(numel, 3, 4096, out, 8);
    CHECK(n == 5);
    CHECK(out[0] == 0 && out[1] == 0 && out[2] == 4096);
    CHECK(out[6] == 0 && out[7] == 8192 && out[8] == 10000 - 8192);
    CHECK(out[9] == 1 && out[10] == 0 && out[11] == 5);
    CHECK(desloc_plan_chunks(NULL, 3, 4096, out, 8) == DESLOC_E_NULL);

    CHECK(strcmp(desloc_strerror(DESLOC_OK), "ok") == 0);
    CHECK(desloc_strerror(-12345) != NULL);

    /* argument errors are reported before any CUDA call */
    desloc_ctx *ctx = (desloc_ctx *)0x1;
    float *ptrs[6] = {0};
    CHECK(desloc_create(&ctx, &cfg, ptrs, ptrs, ptrs, 0) == DESLOC_E_NULL);
    CHECK(ctx == NULL);
    cfg.M = 0;
    CHECK(desloc_create(&ctx, &cfg, ptrs, ptrs, ptrs, 0) == DESLOC_E_RANGE);
    CHECK(desloc_destroy(NULL) == DESLOC_OK);
    CHECK(desloc_step(NULL, 0, 0.f, 0.f, NULL, NULL, NULL) == DESLOC_E_NULL);
    CHECK(sizeof(desloc_config) >= 56);
    printf(fails ? "abi_check: %d failure(s)\n" : "abi_check: ok\n", fails);
    return fails ? 1 : 0;
}
