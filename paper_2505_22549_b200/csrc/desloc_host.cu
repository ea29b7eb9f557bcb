// Host side of the DES-LOC library: the C ABI of include/desloc.h, argument validation, the
// sync schedule (Algorithm 1's "t mod K = 0" tests), the multi-tensor chunk plan and the
// launcher that picks one kernel instantiation per step.  No torch types, no CPU compute path.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <limits>
#include <new>
#include <vector>

#include "../../include/desloc_testing.h"
#include "desloc_inst.cuh"
#include "desloc_internal.cuh"
#include "desloc_norms.cuh"

namespace desloc {

const void *lookup_step_kernel(int opt, bool post, bool bf16, int mt, int mask, bool diag) {
    // A local step (mask 0) is the same code for either ordering and lives in the pre-average
    // units.  Up to MAX_MT workers it uses the all-workers-per-chunk instantiation (more bytes
    // per block and per pointer set-up); beyond that, and for M = 1, workers are separate work
    // items of the local kernel.
    const bool pre = !post || mask == 0;
    const int m = (mask == 0 && !(mt >= 2 && mt <= MAX_MT)) ? 1 : mt;
    if (opt == OPT_ADAM) {
        if (diag) return pre ? lookup_adam_pre_diag(bf16, m, mask) : lookup_adam_post_diag(bf16, m, mask);
        return pre ? lookup_adam_pre(bf16, m, mask) : lookup_adam_post(bf16, m, mask);
    }
    if (opt == OPT_ADOPT) {
        if (diag) return pre ? lookup_adopt_pre_diag(bf16, m, mask) : lookup_adopt_post_diag(bf16, m, mask);
        return pre ? lookup_adopt_pre(bf16, m, mask) : lookup_adopt_post(bf16, m, mask);
    }
    if (opt == OPT_SGDM) {
        if (diag) return pre ? lookup_sgdm_pre_diag(bf16, m, mask) : lookup_sgdm_post_diag(bf16, m, mask);
        return pre ? lookup_sgdm_pre(bf16, m, mask) : lookup_sgdm_post(bf16, m, mask);
    }
    return nullptr;
}

}  // namespace desloc

using desloc::mask_at;
using desloc::validate_config;

namespace {

constexpr int kSlots = 8;  // staging slots for per-step gradient pointer tables
constexpr int kHostGroups = 8;  // pipeline depth of desloc_step_host

struct Slot {
    void **host = nullptr;  // pinned
    void **dev = nullptr;
    cudaEvent_t done = nullptr;
    bool in_flight = false;
};

// desloc_step_host: tensor groups whose copies and kernels are pipelined
struct HostGroup {
    int32_t k0, k1;   // tensors [k0, k1)
    int64_t c0, c1;   // tiles   [c0, c1)
};

// Everything that depends on the worker count M (re-made by desloc_set_workers): the pointer
// tables, the tile plan (the tile length is a function of M) and the scratch sized by either.
struct WorkerRes {
    desloc::Chunk *d_chunks = nullptr;   // tiles of the step kernels
    int64_t nchunks = 0;
    long long *d_tstart = nullptr;       // [num_tensors + 1] first tile of every tensor
    std::vector<HostGroup> groups;
    void **d_tables = nullptr;  // [3][nptr] x, u, v
    Slot slots[kSlots];
    float *d_partial = nullptr;  // reductions: partial sums [2][M][nrchunks]
    float *d_norms = nullptr;    // [3][M]: gradient norms, clip factors, relative change
    void **h_snap = nullptr;     // pinned pointer table for desloc_rel_change
    void **d_snap = nullptr;
    float *d_diag = nullptr;     // diagnostics step: [3][M][nchunks] per-chunk sums of squares
    double *d_diag_sums = nullptr;  // [3][M][num_tensors]
    float *d_diag_out = nullptr;    // [3][M][num_tensors] per-tensor norms, then [3][M] totals
};

void free_worker_res(WorkerRes &r) {
    for (Slot &s : r.slots) {
        if (s.done) cudaEventDestroy(s.done);
        if (s.host) cudaFreeHost(s.host);
        if (s.dev) cudaFree(s.dev);
        s = Slot();
    }
    if (r.d_chunks) cudaFree(r.d_chunks);
    if (r.d_tstart) cudaFree(r.d_tstart);
    if (r.d_tables) cudaFree(r.d_tables);
    if (r.d_partial) cudaFree(r.d_partial);
    if (r.d_norms) cudaFree(r.d_norms);
    if (r.h_snap) cudaFreeHost(r.h_snap);
    if (r.d_snap) cudaFree(r.d_snap);
    if (r.d_diag) cudaFree(r.d_diag);
    if (r.d_diag_sums) cudaFree(r.d_diag_sums);
    if (r.d_diag_out) cudaFree(r.d_diag_out);
    r = WorkerRes();
}

// Allocates and fills the M-dependent resources; the device must be current.  May throw
// std::bad_alloc (host vectors).
cudaError_t make_worker_res(WorkerRes &r, int M, const int64_t *numel, int num_tensors, int64_t total,
                            int64_t nrchunks, bool has_v, float *const *x, float *const *u,
                            float *const *v) {
    // tile plan for this worker count
    const int64_t chunk_elems = desloc::chunk_elems_for(M, numel, num_tensors);
    std::vector<int64_t> heads(static_cast<size_t>(num_tensors));
    for (int32_t k = 0; k < num_tensors; ++k) heads[k] = desloc::head_elems(x[k], numel[k]);
    const int64_t nchunks = desloc::count_chunks(numel, num_tensors, chunk_elems, heads.data());
    std::vector<desloc::Chunk> chunks(static_cast<size_t>(nchunks));
    desloc::fill_chunks(numel, num_tensors, chunk_elems, chunks.data(), heads.data());
    std::vector<long long> tstart(static_cast<size_t>(num_tensors) + 1, 0);
    r.groups.clear();
    {
        // tensor groups of about equal size for desloc_step_host
        int64_t acc = 0, c0 = 0;
        int32_t k0 = 0;
        for (int32_t k = 0; k < num_tensors; ++k) {
            tstart[k + 1] = tstart[k] + desloc::chunks_of(numel[k], chunk_elems, heads[k]);
            acc += numel[k];
            const int done_groups = static_cast<int>(r.groups.size());
            const bool last = k == num_tensors - 1;
            if (last || (done_groups < kHostGroups - 1 && acc * kHostGroups >= total * (done_groups + 1))) {
                r.groups.push_back({k0, k + 1, c0, tstart[k + 1]});
                k0 = k + 1;
                c0 = tstart[k + 1];
            }
        }
    }
    r.nchunks = nchunks;
    cudaError_t e0 = cudaMalloc(&r.d_chunks, chunks.size() * sizeof(desloc::Chunk));
    if (e0 == cudaSuccess)
        e0 = cudaMemcpy(r.d_chunks, chunks.data(), chunks.size() * sizeof(desloc::Chunk), cudaMemcpyHostToDevice);
    if (e0 == cudaSuccess) e0 = cudaMalloc(&r.d_tstart, tstart.size() * sizeof(long long));
    if (e0 == cudaSuccess)
        e0 = cudaMemcpy(r.d_tstart, tstart.data(), tstart.size() * sizeof(long long), cudaMemcpyHostToDevice);
    if (e0 != cudaSuccess) return e0;

    const int64_t nptr = static_cast<int64_t>(M) * num_tensors;
    std::vector<void *> tables(static_cast<size_t>(3 * nptr), nullptr);
    for (int64_t i = 0; i < nptr; ++i) {
        tables[i] = x[i];
        tables[nptr + i] = u[i];
        tables[2 * nptr + i] = has_v ? static_cast<void *>(v[i]) : nullptr;
    }
    cudaError_t e = cudaMalloc(&r.d_tables, tables.size() * sizeof(void *));
    if (e == cudaSuccess)
        e = cudaMemcpy(r.d_tables, tables.data(), tables.size() * sizeof(void *), cudaMemcpyHostToDevice);
    const size_t npart = static_cast<size_t>(2) * M * static_cast<size_t>(nrchunks);
    if (e == cudaSuccess) e = cudaMalloc(&r.d_partial, npart * sizeof(float));
    if (e == cudaSuccess) e = cudaMalloc(&r.d_norms, static_cast<size_t>(3) * M * sizeof(float));
    if (e == cudaSuccess) e = cudaMemset(r.d_norms, 0, static_cast<size_t>(3) * M * sizeof(float));
    if (e == cudaSuccess) e = cudaMallocHost(&r.h_snap, static_cast<size_t>(nptr) * sizeof(void *));
    if (e == cudaSuccess) e = cudaMalloc(&r.d_snap, static_cast<size_t>(nptr) * sizeof(void *));
    const size_t ndiag = static_cast<size_t>(desloc::DIAG_KINDS) * M;
    if (e == cudaSuccess) e = cudaMalloc(&r.d_diag, ndiag * static_cast<size_t>(nchunks) * sizeof(float));
    if (e == cudaSuccess) e = cudaMalloc(&r.d_diag_sums, ndiag * num_tensors * sizeof(double));
    if (e == cudaSuccess) e = cudaMalloc(&r.d_diag_out, ndiag * (num_tensors + 1) * sizeof(float));
    for (int i = 0; i < kSlots && e == cudaSuccess; ++i) {
        Slot &s = r.slots[i];
        e = cudaMallocHost(&s.host, static_cast<size_t>(nptr) * sizeof(void *));
        if (e == cudaSuccess) e = cudaMalloc(&s.dev, static_cast<size_t>(nptr) * sizeof(void *));
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming);
    }
    return e;
}

}  // namespace

struct desloc_ctx {
    desloc_config cfg{};
    std::vector<int64_t> numel;
    int device = 0;
    int64_t total_elems = 0;
    int64_t nptr = 0;  // M * num_tensors
    desloc::Chunk *d_rchunks = nullptr;  // 4096-element chunks of the reduction kernels
    int64_t nrchunks = 0;
    int *h_err = nullptr;                // mapped pinned flag: a device-side wait ran out
    int *d_err = nullptr;                // the same flag as the kernels address it
    int wait_limit = desloc::DEFAULT_WAIT_LIMIT;
    WorkerRes res;
    int next_slot = 0;
    int cur_slot = -1;           // slot holding the table equal to last_grads
    std::vector<const void *> last_grads;
    cudaStream_t last_stream = nullptr;
    int64_t counters[4] = {0, 0, 0, 0};
    int64_t launches = 0;
    int last_cuda_error = 0;
    bool diag_valid = false;        // a diagnostics step has run since the workers last changed
    int64_t max_blocks = 0;         // test hook: cap on the grid (0 = one block per work item)
    int staging_mode = -1;          // test hook: -1 the library decides, 0 always stage, 1 never
    std::vector<const void *> prepared;  // kernels whose shared-memory limit this context has raised
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t ev_entry = nullptr;
    cudaEvent_t ev_group[kHostGroups] = {};
};

namespace {

int cuda_fail(desloc_ctx *ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda_error = static_cast<int>(e);
    (void)cudaGetLastError();  // clear the sticky per-thread error where it can be cleared
    return DESLOC_E_CUDA;
}

void free_ctx(desloc_ctx *ctx) {
    if (!ctx) return;
    free_worker_res(ctx->res);
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    if (ctx->ev_entry) cudaEventDestroy(ctx->ev_entry);
    for (cudaEvent_t ev : ctx->ev_group)
        if (ev) cudaEventDestroy(ev);
    if (ctx->d_rchunks) cudaFree(ctx->d_rchunks);
    if (ctx->h_err) cudaFreeHost(ctx->h_err);
    delete ctx;
}

// Stage the gradient pointer table for this step on `stream`; returns the device table.
int stage_grads(desloc_ctx *ctx, const void *const *grads, cudaStream_t stream, void ***dev_out) {
    const size_t bytes = static_cast<size_t>(ctx->nptr) * sizeof(void *);
    if (ctx->cur_slot >= 0 && stream == ctx->last_stream &&
        std::memcmp(ctx->last_grads.data(), grads, bytes) == 0) {
        *dev_out = ctx->res.slots[ctx->cur_slot].dev;  // same pointers as last step: table is resident
        return DESLOC_OK;
    }
    Slot &s = ctx->res.slots[ctx->next_slot];
    if (s.in_flight) {
        // Re-use of a slot whose kernel was enqueued kSlots table changes ago: wait for it.
        cudaError_t e = cudaEventSynchronize(s.done);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        s.in_flight = false;
    }
    std::memcpy(s.host, grads, bytes);
    cudaError_t e = cudaMemcpyAsync(s.dev, s.host, bytes, cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    std::memcpy(ctx->last_grads.data(), grads, bytes);
    ctx->cur_slot = ctx->next_slot;
    ctx->next_slot = (ctx->next_slot + 1) % kSlots;
    ctx->last_stream = stream;
    *dev_out = s.dev;
    return DESLOC_OK;
}

// max_norm > 0: norm-based clipping first (two reduction launches), then the step.
// diag: the step kernel also accumulates the per-chunk sums of squares of g, x_{t+1} and d_t.
// host_grads != nullptr: the gradients are first copied from host memory into `grads` (device),
// tensor group by tensor group on the context's copy stream, each group's kernel starting as
// soon as its copies have landed.
int run_step(desloc_ctx *ctx, uint32_t mask, float lr_t, float clip_bound_t,
             const void *const *grads, cudaStream_t stream, float max_norm = 0.f,
             const void *const *host_grads = nullptr, bool diag = false) {
    const desloc_config &c = ctx->cfg;
    if (std::isnan(max_norm)) return DESLOC_E_RANGE;
    int rc = desloc::validate_step(&c, lr_t, clip_bound_t);
    if (rc != DESLOC_OK) return rc;
    for (int64_t i = 0; i < ctx->nptr; ++i)
        if (!grads[i]) return DESLOC_E_NULL;
    // a block of an earlier step gave up waiting for its tile: that step is incomplete
    if (*static_cast<volatile int *>(ctx->h_err) != 0) return DESLOC_E_DEVICE_WAIT;

    int dev_before = -1;
    cudaError_t e = cudaGetDevice(&dev_before);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (dev_before != ctx->device) {
        e = cudaSetDevice(ctx->device);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    do {
        // Under stream capture nothing may be staged through the pinned ring (a replay would
        // read whatever the ring holds by then) and no event of the ring may be recorded.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        e = cudaStreamIsCapturing(stream, &cap);
        if (e != cudaSuccess) {
            rc = cuda_fail(ctx, e);
            break;
        }
        const bool capturing = cap != cudaStreamCaptureStatusNone;
        if (capturing && host_grads) {
            rc = DESLOC_E_INVALID;
            break;
        }
        void **d_g = nullptr;
        bool inline_g = false;
        if (!capturing) {
            rc = stage_grads(ctx, grads, stream, &d_g);
            if (rc != DESLOC_OK) break;
        } else if (ctx->nptr <= desloc::INLINE_PTRS && max_norm <= 0.f) {
            inline_g = true;  // pointers travel in the kernel parameters: nothing to keep alive
        } else if (ctx->cur_slot >= 0 && stream == ctx->last_stream &&
                   std::memcmp(ctx->last_grads.data(), grads,
                               static_cast<size_t>(ctx->nptr) * sizeof(void *)) == 0) {
            d_g = ctx->res.slots[ctx->cur_slot].dev;  // table already resident in this slot
        } else {
            rc = DESLOC_E_INVALID;  // stage these pointers with one un-captured step first
            break;
        }
        const float *d_gscale = nullptr;
        if (max_norm > 0.f) {
            e = desloc::launch_grad_norms(ctx->d_rchunks, ctx->nrchunks,
                                          reinterpret_cast<const void *const *>(d_g), c.num_tensors,
                                          c.M, c.grad_dtype == DESLOC_BF16, max_norm,
                                          ctx->res.d_partial, ctx->res.d_norms, ctx->res.d_norms + c.M,
                                          ctx->d_err, ctx->wait_limit, stream);
            if (e != cudaSuccess) {
                rc = cuda_fail(ctx, e);
                break;
            }
            ctx->launches += 2;
            d_gscale = ctx->res.d_norms + c.M;
        }

        const desloc::LaunchPlan plan = desloc::plan_launch(c, mask, ctx->res.nchunks, diag);
        if (!plan.fn) {
            rc = DESLOC_E_INVALID;
            break;
        }
        desloc::StepArgs a{};
        a.chunks = ctx->res.d_chunks;
        a.nchunks = ctx->res.nchunks;
        a.x = reinterpret_cast<float *const *>(ctx->res.d_tables);
        a.u = reinterpret_cast<float *const *>(ctx->res.d_tables + ctx->nptr);
        a.v = reinterpret_cast<float *const *>(ctx->res.d_tables + 2 * ctx->nptr);
        a.g = reinterpret_cast<const void *const *>(d_g);
        if (inline_g)
            for (int64_t i = 0; i < ctx->nptr; ++i) a.g_inline[i] = grads[i];
        a.gscale = d_gscale;
        a.diag = diag ? ctx->res.d_diag : nullptr;
        a.diag_stride = ctx->res.nchunks;
        a.diag_chunk0 = 0;
        desloc::fill_hyper(a, c, lr_t, clip_bound_t);
        a.err = ctx->d_err;
        a.wait_limit = ctx->wait_limit;
        a.direct = ctx->staging_mode < 0 ? (plan.direct ? 1 : 0) : ctx->staging_mode;

        void *params[] = {&a};
        const auto capped = [ctx](const desloc::LaunchPlan &lp) {
            const bool cap = lp.strides && ctx->max_blocks > 0 && lp.grid > ctx->max_blocks;
            return static_cast<unsigned>(cap ? ctx->max_blocks : lp.grid);
        };
        // (once per kernel: the attribute call costs a microsecond that a latency-bound step notices)
        if (std::find(ctx->prepared.begin(), ctx->prepared.end(), plan.fn) == ctx->prepared.end()) {
            e = desloc::prepare_launch(plan);
            if (e != cudaSuccess) {
                rc = cuda_fail(ctx, e);
                break;
            }
            if (ctx->prepared.size() < ctx->prepared.capacity()) ctx->prepared.push_back(plan.fn);
        }
        if (!host_grads) {
            e = cudaLaunchKernel(plan.fn, dim3(capped(plan)),
                                 dim3(desloc::BLOCK_THREADS), params, plan.smem, stream);
            if (e == cudaSuccess) ctx->launches += 1;
        } else {
            // The device gradient buffers may still be read by earlier work on `stream`.
            const size_t gsz = c.grad_dtype == DESLOC_BF16 ? 2 : 4;
            e = cudaEventRecord(ctx->ev_entry, stream);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_stream, ctx->ev_entry, 0);
            for (size_t gi = 0; gi < ctx->res.groups.size() && e == cudaSuccess; ++gi) {
                const HostGroup &grp = ctx->res.groups[gi];
                for (int m = 0; m < c.M && e == cudaSuccess; ++m) {
                    // merge tensors that are adjacent on both sides into one copy
                    int32_t k = grp.k0;
                    while (k < grp.k1 && e == cudaSuccess) {
                        const int64_t i0 = static_cast<int64_t>(m) * c.num_tensors + k;
                        const char *hp = static_cast<const char *>(host_grads[i0]);
                        char *dp = static_cast<char *>(const_cast<void *>(grads[i0]));
                        size_t bytes = static_cast<size_t>(ctx->numel[k]) * gsz;
                        int32_t k2 = k + 1;
                        while (k2 < grp.k1) {
                            const int64_t i2 = static_cast<int64_t>(m) * c.num_tensors + k2;
                            if (static_cast<const char *>(host_grads[i2]) != hp + bytes ||
                                static_cast<const char *>(grads[i2]) != dp + bytes)
                                break;
                            bytes += static_cast<size_t>(ctx->numel[k2]) * gsz;
                            ++k2;
                        }
                        e = cudaMemcpyAsync(dp, hp, bytes, cudaMemcpyHostToDevice, ctx->copy_stream);
                        k = k2;
                    }
                }
                if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_group[gi], ctx->copy_stream);
                if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ctx->ev_group[gi], 0);
                if (e != cudaSuccess) break;
                a.chunks = ctx->res.d_chunks + grp.c0;
                a.nchunks = grp.c1 - grp.c0;
                a.diag_chunk0 = grp.c0;
                const desloc::LaunchPlan gp = desloc::plan_launch(c, mask, a.nchunks, diag);
                e = cudaLaunchKernel(gp.fn, dim3(capped(gp)),
                                     dim3(desloc::BLOCK_THREADS), params, gp.smem, stream);
                if (e == cudaSuccess) ctx->launches += 1;
            }
        }
        if (e != cudaSuccess) {
            rc = cuda_fail(ctx, e);
            break;
        }
        if (!capturing) {
            Slot &s = ctx->res.slots[ctx->cur_slot];
            e = cudaEventRecord(s.done, stream);
            if (e != cudaSuccess) {
                rc = cuda_fail(ctx, e);
                break;
            }
            s.in_flight = true;
        }
        if (diag) ctx->diag_valid = true;
        ctx->counters[0] += 1;
        ctx->counters[1] += (mask & DESLOC_SYNC_X) ? 1 : 0;
        ctx->counters[2] += (mask & DESLOC_SYNC_U) ? 1 : 0;
        ctx->counters[3] += (mask & DESLOC_SYNC_V) ? 1 : 0;
    } while (false);
    if (dev_before != ctx->device) cudaSetDevice(dev_before);
    return rc;
}

}  // namespace

extern "C" {

uint32_t desloc_sync_mask(const desloc_config *cfg, int64_t t) {
    if (!cfg || t < 0) return 0;
    return mask_at(cfg, t);
}

int64_t desloc_chunk_elems(const desloc_config *cfg) {
    if (!cfg || !cfg->numel) return DESLOC_E_NULL;
    if (cfg->M < 1 || cfg->M > DESLOC_MAX_M || cfg->num_tensors < 1) return DESLOC_E_RANGE;
    for (int32_t k = 0; k < cfg->num_tensors; ++k)
        if (cfg->numel[k] < 1) return DESLOC_E_RANGE;
    return desloc::chunk_elems_for(cfg->M, cfg->numel, cfg->num_tensors);
}

int64_t desloc_plan_chunks_at(const int64_t *numel, int32_t num_tensors, int64_t chunk_elems,
                              const void *const *x0, int64_t *out, int64_t cap) {
    if (!numel) return DESLOC_E_NULL;
    if (num_tensors < 1 || chunk_elems < 1 || cap < 0) return DESLOC_E_RANGE;
    if (cap > 0 && !out) return DESLOC_E_NULL;
    for (int32_t k = 0; k < num_tensors; ++k)
        if (numel[k] < 1) return DESLOC_E_RANGE;
    try {
        // the context's own planner, so that this is the table a context works from
        std::vector<int64_t> heads(static_cast<size_t>(num_tensors), 0);
        if (x0)
            for (int32_t k = 0; k < num_tensors; ++k) heads[k] = desloc::head_elems(x0[k], numel[k]);
        const int64_t n = desloc::count_chunks(numel, num_tensors, chunk_elems, heads.data());
        if (cap > 0) {
            std::vector<desloc::Chunk> chunks(static_cast<size_t>(n));
            desloc::fill_chunks(numel, num_tensors, chunk_elems, chunks.data(), heads.data());
            for (int64_t c = 0; c < n && c < cap; ++c) {
                out[3 * c + 0] = chunks[c].tensor;
                out[3 * c + 1] = chunks[c].start;
                out[3 * c + 2] = chunks[c].count;
            }
        }
        return n;
    } catch (const std::bad_alloc &) {
        return DESLOC_E_NOMEM;
    }
}

int64_t desloc_plan_chunks(const int64_t *numel, int32_t num_tensors, int64_t chunk_elems,
                           int64_t *out, int64_t cap) {
    return desloc_plan_chunks_at(numel, num_tensors, chunk_elems, nullptr, out, cap);
}

int desloc_create(desloc_ctx **out, const desloc_config *cfg, float *const *x, float *const *u,
                  float *const *v, int cuda_device) {
    if (!out) return DESLOC_E_NULL;
    *out = nullptr;
    int rc = validate_config(cfg);
    if (rc != DESLOC_OK) return rc;
    if (!cfg->numel || !x || !u) return DESLOC_E_NULL;
    if (cfg->opt != DESLOC_SGDM && !v) return DESLOC_E_NULL;
    if (cuda_device < 0) return DESLOC_E_RANGE;
    const int64_t nptr = static_cast<int64_t>(cfg->M) * cfg->num_tensors;
    int64_t total = 0;
    rc = desloc::validate_numel(cfg, &total);
    if (rc != DESLOC_OK) return rc;
    for (int64_t i = 0; i < nptr; ++i) {
        if (!x[i] || !u[i]) return DESLOC_E_NULL;
        if (cfg->opt != DESLOC_SGDM && !v[i]) return DESLOC_E_NULL;
    }
    // (the reduction kernels' chunks start with the tensors: cutting them at 2 KB boundaries like
    // the step kernels' made no measurable difference, and this way the norms do not depend on
    // where the buffers are)
    const int64_t nrchunks = desloc::count_chunks(cfg->numel, cfg->num_tensors, desloc::REDUCE_CHUNK_ELEMS);
    if (!desloc::grid_fits(cfg->M, cfg->numel, cfg->num_tensors)) return DESLOC_E_RANGE;

    desloc_ctx *ctx = new (std::nothrow) desloc_ctx();
    if (!ctx) return DESLOC_E_NOMEM;
    std::vector<desloc::Chunk> rchunks;
    try {
        ctx->numel.assign(cfg->numel, cfg->numel + cfg->num_tensors);
        ctx->last_grads.assign(static_cast<size_t>(nptr), nullptr);
        ctx->prepared.reserve(64);   // steps never allocate: beyond this the attribute is simply set again
        rchunks.resize(static_cast<size_t>(nrchunks));
        desloc::fill_chunks(cfg->numel, cfg->num_tensors, desloc::REDUCE_CHUNK_ELEMS, rchunks.data());
    } catch (const std::bad_alloc &) {
        delete ctx;
        return DESLOC_E_NOMEM;
    }
    ctx->cfg = *cfg;
    ctx->cfg.numel = ctx->numel.data();
    ctx->device = cuda_device;
    ctx->total_elems = total;
    ctx->nptr = nptr;
    ctx->nrchunks = nrchunks;

    int dev_before = -1;
    cudaError_t e = cudaGetDevice(&dev_before);
    if (e == cudaSuccess && dev_before != cuda_device) e = cudaSetDevice(cuda_device);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_rchunks, rchunks.size() * sizeof(desloc::Chunk));
    if (e == cudaSuccess)
        e = cudaMemcpy(ctx->d_rchunks, rchunks.data(), rchunks.size() * sizeof(desloc::Chunk),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaHostAlloc(reinterpret_cast<void **>(&ctx->h_err), sizeof(int), cudaHostAllocMapped);
    if (e == cudaSuccess) {
        *ctx->h_err = 0;
        e = cudaHostGetDevicePointer(reinterpret_cast<void **>(&ctx->d_err), ctx->h_err, 0);
    }
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_entry, cudaEventDisableTiming);
    for (int i = 0; i < kHostGroups && e == cudaSuccess; ++i)
        e = cudaEventCreateWithFlags(&ctx->ev_group[i], cudaEventDisableTiming);
    if (e == cudaSuccess) {
        try {
            e = make_worker_res(ctx->res, cfg->M, ctx->numel.data(), cfg->num_tensors, total, nrchunks,
                                cfg->opt != DESLOC_SGDM, x, u, v);
        } catch (const std::bad_alloc &) {
            e = cudaErrorMemoryAllocation;
        }
    }
    if (dev_before >= 0 && dev_before != cuda_device) cudaSetDevice(dev_before);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        free_ctx(ctx);
        return e == cudaErrorMemoryAllocation ? DESLOC_E_NOMEM : DESLOC_E_CUDA;
    }
    *out = ctx;
    return DESLOC_OK;
}

int desloc_step(desloc_ctx *ctx, int64_t t, float lr_t, float clip_bound_t,
                const void *const *grads, void *stream, uint32_t *mask_out) {
    desloc::NvtxRange range("desloc_step");
    if (!ctx || !grads) return DESLOC_E_NULL;
    if (t < 0) return DESLOC_E_RANGE;
    const uint32_t mask = mask_at(&ctx->cfg, t);
    const int rc = run_step(ctx, mask, lr_t, clip_bound_t, grads, static_cast<cudaStream_t>(stream));
    if (rc == DESLOC_OK && mask_out) *mask_out = mask;
    return rc;
}

int desloc_step_diag(desloc_ctx *ctx, int64_t t, float lr_t, float clip_bound_t, float max_norm,
                     const void *const *grads, void *stream, uint32_t *mask_out) {
    desloc::NvtxRange range("desloc_step_diag");
    if (!ctx || !grads) return DESLOC_E_NULL;
    if (t < 0 || !(max_norm >= 0.f) || !std::isfinite(max_norm)) return DESLOC_E_RANGE;
    const uint32_t mask = mask_at(&ctx->cfg, t);
    const int rc = run_step(ctx, mask, lr_t, clip_bound_t, grads, static_cast<cudaStream_t>(stream),
                            max_norm, nullptr, true);
    if (rc == DESLOC_OK && mask_out) *mask_out = mask;
    return rc;
}

int desloc_get_diag_norms(desloc_ctx *ctx, float *per_tensor_out, float *total_out, void *stream) {
    if (!ctx) return DESLOC_E_NULL;
    if (!ctx->diag_valid) return DESLOC_E_INVALID;
    const desloc_config &c = ctx->cfg;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev_before = -1;
    cudaError_t e = cudaGetDevice(&dev_before);
    if (e == cudaSuccess && dev_before != ctx->device) e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    const size_t rows = static_cast<size_t>(desloc::DIAG_KINDS) * c.M;
    float *d_per = ctx->res.d_diag_out, *d_tot = ctx->res.d_diag_out + rows * c.num_tensors;
    e = desloc::launch_diag_norms(ctx->res.d_diag, ctx->res.nchunks, ctx->res.d_tstart, c.num_tensors, c.M,
                                  ctx->res.d_diag_sums, d_per, d_tot, st);
    if (e == cudaSuccess) {
        ctx->launches += 2;
        if (per_tensor_out)
            e = cudaMemcpyAsync(per_tensor_out, d_per, rows * c.num_tensors * sizeof(float),
                                cudaMemcpyDeviceToHost, st);
    }
    if (e == cudaSuccess && total_out)
        e = cudaMemcpyAsync(total_out, d_tot, rows * sizeof(float), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (dev_before != ctx->device) cudaSetDevice(dev_before);
    return e == cudaSuccess ? DESLOC_OK : cuda_fail(ctx, e);
}

int desloc_step_host(desloc_ctx *ctx, int64_t t, float lr_t, float clip_bound_t,
                     const void *const *host_grads, void *const *dev_grads, void *stream,
                     uint32_t *mask_out) {
    desloc::NvtxRange range("desloc_step_host");
    if (!ctx || !host_grads || !dev_grads) return DESLOC_E_NULL;
    if (t < 0) return DESLOC_E_RANGE;
    for (int64_t i = 0; i < ctx->nptr; ++i)
        if (!host_grads[i]) return DESLOC_E_NULL;
    const uint32_t mask = mask_at(&ctx->cfg, t);
    const int rc = run_step(ctx, mask, lr_t, clip_bound_t,
                            reinterpret_cast<const void *const *>(dev_grads),
                            static_cast<cudaStream_t>(stream), 0.f, host_grads);
    if (rc == DESLOC_OK && mask_out) *mask_out = mask;
    return rc;
}

int desloc_step_masked(desloc_ctx *ctx, uint32_t mask, float lr_t, float clip_bound_t,
                       const void *const *grads, void *stream) {
    desloc::NvtxRange range("desloc_step_masked");
    if (!ctx || !grads) return DESLOC_E_NULL;
    if (mask & ~7u) return DESLOC_E_INVALID;
    if (ctx->cfg.opt == DESLOC_SGDM && (mask & DESLOC_SYNC_V)) return DESLOC_E_INVALID;
    return run_step(ctx, mask, lr_t, clip_bound_t, grads, static_cast<cudaStream_t>(stream));
}

int desloc_step_normclip(desloc_ctx *ctx, int64_t t, float lr_t, float clip_bound_t,
                         float max_norm, const void *const *grads, void *stream,
                         uint32_t *mask_out) {
    desloc::NvtxRange range("desloc_step_normclip");
    if (!ctx || !grads) return DESLOC_E_NULL;
    if (t < 0 || !(max_norm > 0.f) || !std::isfinite(max_norm)) return DESLOC_E_RANGE;
    const uint32_t mask = mask_at(&ctx->cfg, t);
    const int rc = run_step(ctx, mask, lr_t, clip_bound_t, grads, static_cast<cudaStream_t>(stream),
                            max_norm);
    if (rc == DESLOC_OK && mask_out) *mask_out = mask;
    return rc;
}

int desloc_get_grad_norms(desloc_ctx *ctx, float *norms_out, float *scales_out, void *stream) {
    if (!ctx) return DESLOC_E_NULL;
    const size_t bytes = static_cast<size_t>(ctx->cfg.M) * sizeof(float);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev_before = -1;
    cudaError_t e = cudaGetDevice(&dev_before);
    if (e == cudaSuccess && dev_before != ctx->device) e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (norms_out) e = cudaMemcpyAsync(norms_out, ctx->res.d_norms, bytes, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && scales_out)
        e = cudaMemcpyAsync(scales_out, ctx->res.d_norms + ctx->cfg.M, bytes, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (dev_before != ctx->device) cudaSetDevice(dev_before);
    return e == cudaSuccess ? DESLOC_OK : cuda_fail(ctx, e);
}

int desloc_rel_change(desloc_ctx *ctx, int32_t array, const float *const *then, float *out,
                      void *stream) {
    if (!ctx || !then || !out) return DESLOC_E_NULL;
    if (array < 0 || array > 2 || (array == 2 && ctx->cfg.opt == DESLOC_SGDM)) return DESLOC_E_INVALID;
    for (int64_t i = 0; i < ctx->nptr; ++i)
        if (!then[i]) return DESLOC_E_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev_before = -1;
    cudaError_t e = cudaGetDevice(&dev_before);
    if (e == cudaSuccess && dev_before != ctx->device) e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    const size_t tbytes = static_cast<size_t>(ctx->nptr) * sizeof(void *);
    // The call ends with a stream synchronisation, so the pinned table is free again on return.
    std::memcpy(ctx->res.h_snap, then, tbytes);
    e = cudaMemcpyAsync(ctx->res.d_snap, ctx->res.h_snap, tbytes, cudaMemcpyHostToDevice, st);
    float *d_out = ctx->res.d_norms + 2 * ctx->cfg.M;
    if (e == cudaSuccess)
        e = desloc::launch_rel_change(
            ctx->d_rchunks, ctx->nrchunks,
            reinterpret_cast<const float *const *>(ctx->res.d_tables + array * ctx->nptr),
            reinterpret_cast<const float *const *>(ctx->res.d_snap), ctx->cfg.num_tensors, ctx->cfg.M,
            ctx->res.d_partial, d_out, st);
    if (e == cudaSuccess) {
        ctx->launches += 2;
        e = cudaMemcpyAsync(out, d_out, static_cast<size_t>(ctx->cfg.M) * sizeof(float),
                            cudaMemcpyDeviceToHost, st);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (dev_before != ctx->device) cudaSetDevice(dev_before);
    return e == cudaSuccess ? DESLOC_OK : cuda_fail(ctx, e);
}

int desloc_set_workers(desloc_ctx *ctx, int32_t M_new, int32_t first_new, float *const *x,
                       float *const *u, float *const *v, void *stream) {
    if (!ctx || !x || !u) return DESLOC_E_NULL;
    const bool has_v = ctx->cfg.opt != DESLOC_SGDM;
    if (has_v && !v) return DESLOC_E_NULL;
    if (M_new < 1 || M_new > DESLOC_MAX_M || first_new < 0 || first_new > M_new) return DESLOC_E_RANGE;
    if (!desloc::grid_fits(M_new, ctx->numel.data(), ctx->cfg.num_tensors)) return DESLOC_E_RANGE;
    const int nt = ctx->cfg.num_tensors;
    const int64_t nptr_new = static_cast<int64_t>(M_new) * nt;
    for (int64_t i = 0; i < nptr_new; ++i) {
        if (!x[i] || !u[i] || (has_v && !v[i])) return DESLOC_E_NULL;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev_before = -1;
    cudaError_t e = cudaGetDevice(&dev_before);
    if (e == cudaSuccess && dev_before != ctx->device) e = cudaSetDevice(ctx->device);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    // Earlier steps must have finished with the old tables before they are replaced.
    e = cudaStreamSynchronize(st);
    WorkerRes fresh;
    if (e == cudaSuccess) {
        try {
            e = make_worker_res(fresh, M_new, ctx->numel.data(), nt, ctx->total_elems, ctx->nrchunks, has_v, x, u, v);
            if (ctx->last_grads.capacity() < static_cast<size_t>(nptr_new))
                ctx->last_grads.reserve(static_cast<size_t>(nptr_new));  // may throw; no state changed yet
        } catch (const std::bad_alloc &) {
            e = cudaErrorMemoryAllocation;
        }
    }
    const int n_new = M_new - first_new;
    if (e == cudaSuccess && n_new > 0) {
        // New replicas start from the mean of ALL replicas the context held so far.
        const int n_arr = has_v ? 3 : 2;
        for (int arr = 0; arr < n_arr && e == cudaSuccess; ++arr)
            e = desloc::launch_mean_fill(
                ctx->d_rchunks, ctx->nrchunks,
                reinterpret_cast<const float *const *>(ctx->res.d_tables + arr * ctx->nptr), ctx->cfg.M,
                reinterpret_cast<float *const *>(fresh.d_tables + arr * nptr_new +
                                                 static_cast<int64_t>(first_new) * nt),
                n_new, nt, st);
        if (e == cudaSuccess) ctx->launches += n_arr;
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    int rc = DESLOC_OK;
    if (e == cudaSuccess) {
        free_worker_res(ctx->res);
        ctx->res = fresh;
        ctx->last_grads.assign(static_cast<size_t>(nptr_new), nullptr);  // capacity reserved above
        ctx->cfg.M = M_new;
        ctx->nptr = nptr_new;
        ctx->next_slot = 0;
        ctx->cur_slot = -1;
        ctx->diag_valid = false;
    } else {
        free_worker_res(fresh);
        rc = (e == cudaErrorMemoryAllocation) ? DESLOC_E_NOMEM : cuda_fail(ctx, e);
        (void)cudaGetLastError();
    }
    if (dev_before != ctx->device) cudaSetDevice(dev_before);
    return rc;
}

int desloc_destroy(desloc_ctx *ctx) {
    if (!ctx) return DESLOC_OK;
    int dev_before = -1;
    if (cudaGetDevice(&dev_before) == cudaSuccess && dev_before != ctx->device)
        cudaSetDevice(ctx->device);
    const int device = ctx->device;
    free_ctx(ctx);
    if (dev_before >= 0 && dev_before != device) cudaSetDevice(dev_before);
    (void)cudaGetLastError();
    return DESLOC_OK;
}

int desloc_get_counters(const desloc_ctx *ctx, int64_t out[4]) {
    if (!ctx || !out) return DESLOC_E_NULL;
    for (int i = 0; i < 4; ++i) out[i] = ctx->counters[i];
    return DESLOC_OK;
}

int64_t desloc_get_launch_count(const desloc_ctx *ctx) { return ctx ? ctx->launches : 0; }

int desloc_testing_set_max_blocks(desloc_ctx *ctx, int64_t max_blocks) {
    if (!ctx) return DESLOC_E_NULL;
    if (max_blocks < 0) return DESLOC_E_RANGE;
    ctx->max_blocks = max_blocks;
    return DESLOC_OK;
}

int desloc_testing_set_staging(desloc_ctx *ctx, int32_t mode) {
    if (!ctx) return DESLOC_E_NULL;
    if (mode < -1 || mode > 1) return DESLOC_E_RANGE;
    ctx->staging_mode = mode;
    return DESLOC_OK;
}

int desloc_testing_set_wait_limit(desloc_ctx *ctx, int32_t polls) {
    if (!ctx) return DESLOC_E_NULL;
    ctx->wait_limit = polls < 0 ? desloc::DEFAULT_WAIT_LIMIT : polls;
    if (polls < 0) *static_cast<volatile int *>(ctx->h_err) = 0;
    return DESLOC_OK;
}

int desloc_last_cuda_error(const desloc_ctx *ctx) { return ctx ? ctx->last_cuda_error : 0; }

const char *desloc_strerror(int status) {
    switch (status) {
        case DESLOC_OK: return "ok";
        case DESLOC_E_NULL: return "a required pointer is NULL";
        case DESLOC_E_RANGE: return "argument out of range";
        case DESLOC_E_INVALID: return "invalid optimizer, dtype, flag or mask";
        case DESLOC_E_NOMEM: return "out of memory";
        case DESLOC_E_CUDA: return "CUDA call failed";
        case DESLOC_E_TOO_LARGE: return "problem exceeds the fixed scratch of desloc_step_static";
        case DESLOC_E_DEVICE_WAIT: return "a bounded wait on the device ran out in an earlier step";
        default: return "unknown status";
    }
}

}  // extern "C"
