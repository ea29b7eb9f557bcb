/* A plain C99 program that drives the DES-LOC C ABI on a GPU with nothing but the CUDA runtime:
 * no Python, no torch.  It runs T steps of DES-LOC-Adam for M = 3 workers on a tightly packed
 * tensor list (the third tensor starts at an odd offset) and checks the result against the CPU
 * oracle, which it calls through the oracle library's own C entry point.
 * Exit code 0 = parity within 1e-5 (relative, with the tensor's RMS as floor). */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <cuda_runtime_api.h>

#include "desloc.h"

/* the oracle's configuration record and step routine (oracle/desloc_oracle.c) */
typedef struct {
    int32_t M;
    int32_t opt;
    double beta1, beta2;
    double eps;
    double weight_decay;
    double clip_rho;
    int32_t Kx, Ku, Kv;
    uint32_t flags;
} oracle_cfg;
extern uint32_t desloc_oracle_step(const oracle_cfg *c, int64_t t, double lr, double clip_bound,
                                   int64_t n, int64_t stride, float *x, float *u, float *v,
                                   const float *g);

#define NW 3   /* workers */
#define NT 3
#define T_STEPS 9
static const int64_t numel[NT] = {9000, 777, 5};

static uint64_t rng_state = 0x9E3779B97F4A7C15ull;
static float uniform_pm1(void) {   /* 64-bit LCG, top 24 bits -> [-1, 1) */
    rng_state = rng_state * 6364136223846793005ull + 1442695040888963407ull;
    return (float)((double)(rng_state >> 40) / 8388608.0 - 1.0);
}

#define CUDA_OK(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { \
    printf("CUDA error %s at line %d\n", cudaGetErrorString(e_), __LINE__); return 2; } } while (0)
#define DESLOC_OK_(call) do { int rc_ = (call); if (rc_ != DESLOC_OK) { \
    printf("%s -> %s (line %d)\n", #call, desloc_strerror(rc_), __LINE__); return 3; } } while (0)

/* Steps per second a C caller gets on the latency-bound workload (N = 4096, two workers, fp32
 * gradients, periods 4/8/16): 2000 back-to-back desloc_step() calls between two events.
 * Printed for information, not checked. */
static int eager_latency(void) {
    const int64_t one[1] = {4096};
    float *d;
    CUDA_OK(cudaMalloc((void **)&d, 4 * 2 * 4096 * sizeof(float)));
    CUDA_OK(cudaMemset(d, 0, 4 * 2 * 4096 * sizeof(float)));
    float *x[2] = {d, d + 4096}, *u[2] = {d + 2 * 4096, d + 3 * 4096}, *v[2] = {d + 4 * 4096, d + 5 * 4096};
    const void *g[2] = {d + 6 * 4096, d + 7 * 4096};
    desloc_config cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.M = 2; cfg.num_tensors = 1; cfg.numel = one; cfg.opt = DESLOC_ADAM; cfg.grad_dtype = DESLOC_F32;
    cfg.beta1 = 0.9f; cfg.beta2 = 0.999f; cfg.eps = 1e-8f; cfg.Kx = 4; cfg.Ku = 8; cfg.Kv = 16;
    desloc_ctx *ctx = NULL;
    DESLOC_OK_(desloc_create(&ctx, &cfg, x, u, v, 0));
    cudaEvent_t e0, e1;
    CUDA_OK(cudaEventCreate(&e0));
    CUDA_OK(cudaEventCreate(&e1));
    for (int64_t t = 0; t < 64; ++t) DESLOC_OK_(desloc_step(ctx, t, 1e-3f, 0.f, g, NULL, NULL));
    CUDA_OK(cudaEventRecord(e0, NULL));
    const int steps = 2000;
    for (int64_t t = 64; t < 64 + steps; ++t) DESLOC_OK_(desloc_step(ctx, t, 1e-3f, 0.f, g, NULL, NULL));
    CUDA_OK(cudaEventRecord(e1, NULL));
    CUDA_OK(cudaEventSynchronize(e1));
    float ms = 0.f;
    CUDA_OK(cudaEventElapsedTime(&ms, e0, e1));
    printf("eager desloc_step() from C, N = 4096, M = 2: %.2f us per step\n", 1e3 * ms / steps);
    DESLOC_OK_(desloc_destroy(ctx));
    cudaEventDestroy(e0); cudaEventDestroy(e1); cudaFree(d);
    return 0;
}

int main(void) {
    int64_t off[NT], n = 0;
    for (int k = 0; k < NT; ++k) { off[k] = n; n += numel[k]; }
    const size_t count = (size_t)NW * (size_t)n, bytes = count * sizeof(float);

    float *hx = malloc(bytes), *hu = calloc(count, sizeof(float)), *hv = calloc(count, sizeof(float));
    float *hg = malloc(bytes), *gx = malloc(bytes), *gu = malloc(bytes), *gv = malloc(bytes);
    if (!hx || !hu || !hv || !hg || !gx || !gu || !gv) return 2;
    for (int64_t i = 0; i < n; ++i) {          /* the same start on every worker */
        const float v = 0.02f * uniform_pm1();
        for (int m = 0; m < NW; ++m) hx[(size_t)m * n + i] = v;
    }

    float *dx, *du, *dv, *dg;
    CUDA_OK(cudaSetDevice(0));
    CUDA_OK(cudaMalloc((void **)&dx, bytes));
    CUDA_OK(cudaMalloc((void **)&du, bytes));
    CUDA_OK(cudaMalloc((void **)&dv, bytes));
    CUDA_OK(cudaMalloc((void **)&dg, bytes));
    CUDA_OK(cudaMemcpy(dx, hx, bytes, cudaMemcpyHostToDevice));
    CUDA_OK(cudaMemset(du, 0, bytes));
    CUDA_OK(cudaMemset(dv, 0, bytes));

    float *px[NW * NT], *pu[NW * NT], *pv[NW * NT];
    const void *pg[NW * NT];
    for (int m = 0; m < NW; ++m)
        for (int k = 0; k < NT; ++k) {
            const size_t o = (size_t)m * n + off[k];
            px[m * NT + k] = dx + o; pu[m * NT + k] = du + o; pv[m * NT + k] = dv + o; pg[m * NT + k] = dg + o;
        }

    desloc_config cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.M = NW; cfg.num_tensors = NT; cfg.numel = numel;
    cfg.opt = DESLOC_ADAM; cfg.grad_dtype = DESLOC_F32;
    cfg.beta1 = 0.9f; cfg.beta2 = 0.99f; cfg.eps = 1e-3f; cfg.weight_decay = 0.01f; cfg.clip_rho = 0.75f;
    cfg.Kx = 2; cfg.Ku = 3; cfg.Kv = 4;
    oracle_cfg oc;
    memset(&oc, 0, sizeof oc);
    oc.M = NW; oc.opt = 0;
    oc.beta1 = (double)cfg.beta1; oc.beta2 = (double)cfg.beta2; oc.eps = (double)cfg.eps;
    oc.weight_decay = (double)cfg.weight_decay; oc.clip_rho = (double)cfg.clip_rho;
    oc.Kx = cfg.Kx; oc.Ku = cfg.Ku; oc.Kv = cfg.Kv;

    desloc_ctx *ctx = NULL;
    DESLOC_OK_(desloc_create(&ctx, &cfg, px, pu, pv, 0));
    const float lr = 1e-2f;
    for (int64_t t = 0; t < T_STEPS; ++t) {
        for (size_t i = 0; i < count; ++i) hg[i] = uniform_pm1();
        CUDA_OK(cudaMemcpy(dg, hg, bytes, cudaMemcpyHostToDevice));
        uint32_t mask = 0;
        DESLOC_OK_(desloc_step(ctx, t, lr, 0.f, pg, NULL, &mask));
        const uint32_t want = desloc_oracle_step(&oc, t, (double)lr, 0.0, n, n, hx, hu, hv, hg);
        if (mask != want || mask != desloc_sync_mask(&cfg, t)) {
            printf("step %lld: mask %u, oracle %u\n", (long long)t, mask, want);
            return 1;
        }
        CUDA_OK(cudaDeviceSynchronize());   /* hg is reused for the next step's gradients */
    }
    int64_t counters[4];
    DESLOC_OK_(desloc_get_counters(ctx, counters));
    if (counters[0] != T_STEPS || counters[1] != 5 || counters[2] != 3 || counters[3] != 3) {
        printf("counters %lld %lld %lld %lld\n", (long long)counters[0], (long long)counters[1],
               (long long)counters[2], (long long)counters[3]);
        return 1;
    }
    CUDA_OK(cudaMemcpy(gx, dx, bytes, cudaMemcpyDeviceToHost));
    CUDA_OK(cudaMemcpy(gu, du, bytes, cudaMemcpyDeviceToHost));
    CUDA_OK(cudaMemcpy(gv, dv, bytes, cudaMemcpyDeviceToHost));
    DESLOC_OK_(desloc_destroy(ctx));

    /* max_i |gpu - ref| / max(|ref|, rms(ref tensor)); tensors of fewer than 64 elements take
       the RMS of the worker's whole array as floor */
    const float *got[3] = {gx, gu, gv}, *ref[3] = {hx, hu, hv};
    double worst = 0.0, moved = 0.0;
    for (int a = 0; a < 3; ++a)
        for (int m = 0; m < NW; ++m) {
            double ss_all = 0.0;
            for (int64_t i = 0; i < n; ++i) { const double r = ref[a][(size_t)m * n + i]; ss_all += r * r; }
            const double rms_all = sqrt(ss_all / (double)n);
            for (int k = 0; k < NT; ++k) {
                double ss = 0.0;
                for (int64_t i = 0; i < numel[k]; ++i) { const double r = ref[a][(size_t)m * n + off[k] + i]; ss += r * r; }
                const double floor_ = numel[k] < 64 ? rms_all : sqrt(ss / (double)numel[k]);
                for (int64_t i = 0; i < numel[k]; ++i) {
                    const size_t j = (size_t)m * n + off[k] + i;
                    const double r = ref[a][j], den = fabs(r) > floor_ ? fabs(r) : floor_;
                    const double e = fabs((double)got[a][j] - r) / (den > 1e-30 ? den : 1e-30);
                    if (e > worst) worst = e;
                }
            }
            if (a == 1) moved += ss_all;
        }
    printf("gpu_parity: max relative error %.3e over %zu values x 3 arrays, |u|^2 = %.3e\n", worst, count, moved);
    if (!(moved > 0.0)) { printf("the run did not move the state\n"); return 1; }
    cudaFree(dx); cudaFree(du); cudaFree(dv); cudaFree(dg);
    free(hx); free(hu); free(hv); free(hg); free(gx); free(gu); free(gv);
    if (worst > 1e-5) { printf("gpu_parity: FAILED\n"); return 1; }
    const int rc = eager_latency();
    if (rc) return rc;
    printf("gpu_parity: ok\n");
    return 0;
}
