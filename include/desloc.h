/*
 * desloc.h -- C ABI of the DES-LOC optimizer-step library for NVIDIA B200 (sm_100a).
 *
 * DES-LOC (Desynced Low Communication Adaptive Optimizers): M workers each take
 * local Adam, ADOPT or SGD-momentum steps; the parameters x and the optimizer
 * states u (first moment / momentum) and v (second moment) are averaged across
 * workers on independent periods K_x, K_u, K_v (Algorithm 1 of the paper).
 *
 * This library keeps all M worker replicas in ONE GPU's memory.  One call to
 * desloc_step() runs one step t of Algorithm 1 for all workers: a single
 * memory-bound kernel brings g, x, u, v of every replica on chip once (tile by
 * tile, with bulk asynchronous copies), clips the gradient, averages the arrays
 * whose period divides t (a fixed summation tree over m), applies the
 * per-worker update and writes x, u, v back.
 * A sync step therefore moves the same bytes as a local step; there is no
 * separate averaging pass and no collective.
 *
 * Conventions
 *   - Every pointer named "device" must be valid on the CUDA device given to
 *     desloc_create(); every other pointer is host memory.
 *   - x, u, v are fp32 and caller-owned; the library updates them in place and
 *     borrows the pointers for the lifetime of the context.  Gradients are
 *     fp32 or bf16, read-only, and may live somewhere else at every step.
 *   - All functions return DESLOC_OK (0) or a negative desloc_status; nothing
 *     throws, aborts or prints.  desloc_last_cuda_error() gives the CUDA error
 *     behind a DESLOC_E_CUDA.  There is no CPU fallback: without a usable
 *     device every compute entry point returns DESLOC_E_CUDA.
 *   - One context may be used by one host thread at a time.
 */
#ifndef DESLOC_H_
#define DESLOC_H_

#include <stdint.h>

#if defined(__GNUC__)
#define DESLOC_API __attribute__((visibility("default")))
#else
#define DESLOC_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define DESLOC_MAX_M 256 /* largest worker count a context accepts (the toy problem of the paper uses 256) */

typedef struct desloc_ctx desloc_ctx; /* opaque, library-owned */

typedef enum {
    DESLOC_ADAM = 0,  /* Algorithm 2 */
    DESLOC_ADOPT = 1, /* Algorithm 3 */
    DESLOC_SGDM = 2   /* Algorithm 1 with N = 1 state: u = beta u + (1-beta) g, x = x - eta u */
} desloc_opt_t;

typedef enum { DESLOC_F32 = 0, DESLOC_BF16 = 1 } desloc_dtype_t;

/* Bits of the sync mask: which arrays are averaged over the workers at a step. */
enum { DESLOC_SYNC_X = 1, DESLOC_SYNC_U = 2, DESLOC_SYNC_V = 4 };

enum {
    /* ADOPT only: clamp the normalised gradient g / max(sqrt(v), eps) to +-clip_bound_t,
       the per-step bound handed to desloc_step().  Not part of Algorithm 3; the ADOPT
       optimizer the paper builds on has it, and with v_{-1} = 0 it keeps step 0 finite. */
    DESLOC_FLAG_ADOPT_NORM_CLIP = 1u,
    /* Average AFTER the local update instead of before it (the ordering of Algorithms 4
       and 5): on a sync step the new u / v / x are averaged and every worker stores the mean. */
    DESLOC_FLAG_POST_AVERAGE = 2u
};

typedef enum {
    DESLOC_OK = 0,
    DESLOC_E_NULL = -1,    /* a required pointer is NULL */
    DESLOC_E_RANGE = -2,   /* M, a period, a beta, eps, weight decay, numel or t out of range */
    DESLOC_E_INVALID = -3, /* unknown optimizer / dtype / flag, or a flag the optimizer lacks */
    DESLOC_E_NOMEM = -4,   /* host or device allocation failed */
    DESLOC_E_CUDA = -5,    /* a CUDA call failed; see desloc_last_cuda_error() */
    DESLOC_E_TOO_LARGE = -6, /* desloc_step_static(): the problem exceeds the fixed scratch */
    DESLOC_E_DEVICE_WAIT = -7 /* a thread block of an earlier step gave up waiting for its data
                                 (every wait on the device is bounded): that step is incomplete and
                                 the state undefined; every later step call returns this status */
} desloc_status;

/* The "Require" block of Algorithms 1-3: everything fixed for a run.  Plain data, copied
   by desloc_create(). */
typedef struct {
    int32_t M;              /* workers, 1..DESLOC_MAX_M */
    int32_t num_tensors;    /* >= 1: the model is a list of tensors */
    const int64_t *numel;   /* host, [num_tensors], each >= 1 */
    int32_t opt;            /* desloc_opt_t */
    int32_t grad_dtype;     /* desloc_dtype_t of the gradients */
    float beta1, beta2;     /* decay factors in [0, 1); SGDM uses beta1 only */
    float eps;              /* Adam: lambda, enters as sqrt(v + lambda^2); ADOPT: epsilon in
                               max(sqrt(v), epsilon); >= 0 */
    float weight_decay;     /* >= 0, decoupled: x* (1 - eta_t wd) - d_t.  The paper uses 0. */
    float clip_rho;         /* coordinate clip radius rho of Section 3.1; <= 0 switches it off */
    int32_t Kx, Ku, Kv;     /* sync periods, >= 0; 0 = never (K = infinity); SGDM ignores Kv */
    uint32_t flags;         /* DESLOC_FLAG_* */
} desloc_config;

/*
 * Which arrays Algorithm 1 averages at step t (t counts from 0, so t = 0 syncs every array
 * with a non-zero period): bit X iff Kx > 0 and t mod Kx == 0, likewise U and V; the V bit is
 * always clear for SGDM.  Pure host function; cfg->numel is not read.  Returns 0 for a NULL
 * cfg or t < 0.
 */
DESLOC_API uint32_t desloc_sync_mask(const desloc_config *cfg, int64_t t);

/*
 * Create a context for `cfg` on CUDA device `cuda_device`.
 *   x, u, v : host arrays of M*num_tensors DEVICE pointers, entry [m*num_tensors + k] is worker
 *             m's copy of tensor k (numel[k] fp32 values).  v may be NULL for SGDM.  No two
 *             entries may overlap.  The pointer arrays themselves are copied; the tensors are
 *             borrowed until desloc_destroy().  Any alignment is accepted: tensors whose
 *             pointers are all 16-byte aligned take the vector path, the rest a scalar path.
 * Validates everything before touching the device.  Allocates the context, its device-side
 * pointer and chunk tables, and a few pinned staging buffers -- nothing is allocated later.
 * Initial state is whatever the buffers hold (Algorithm 1 starts every worker from the same
 * x_0 and zero states).
 */
DESLOC_API int desloc_create(desloc_ctx **out, const desloc_config *cfg, float *const *x, float *const *u,
                  float *const *v, int cuda_device);

/*
 * One step t of Algorithm 1 (Algorithm 2 / 3 / SGDM per cfg.opt) for all M workers.
 *   t            : step counter, >= 0; decides the sync mask via desloc_sync_mask().
 *   lr_t         : eta_t, the learning rate of this step (the schedule is the caller's).
 *   clip_bound_t : bound for DESLOC_FLAG_ADOPT_NORM_CLIP at this step; ignored otherwise.
 *   grads        : host array of M*num_tensors DEVICE pointers (same indexing as x) to
 *                  gradients of cfg.grad_dtype; read-only; may differ from call to call.
 *   stream       : a cudaStream_t (NULL = default stream).  The call only enqueues work and
 *                  never synchronises the device.
 *   mask_out     : if not NULL receives the sync mask that was applied.
 * Errors: a failed launch is returned by this call; an asynchronous execution error surfaces
 * in a later call or at the caller's next synchronisation.
 *
 * Stream capture (CUDA graphs, for small launch-bound problems): the call may be made while
 * `stream` is capturing if either M*num_tensors <= 32 (the gradient pointers then travel in
 * the kernel parameters) or `grads` holds the same pointers as the previous, un-captured call
 * on that stream; otherwise it returns DESLOC_E_INVALID and captures nothing.  (In the second
 * case the captured launch refers to the context's staging slot of that pointer set, which is
 * recycled after eight later un-captured calls with other gradient pointers: replay the graph
 * only while fewer than eight such calls have been made.)  t, lr_t and
 * clip_bound_t are frozen into the captured launch, so a replayed graph repeats the same mask
 * sequence: capture a window of lcm(Kx, Ku, Kv) steps starting at a multiple of it.  Counters
 * and the launch count advance when a call is captured, not when the graph is replayed.
 */
DESLOC_API int desloc_step(desloc_ctx *ctx, int64_t t, float lr_t, float clip_bound_t,
                const void *const *grads, void *stream, uint32_t *mask_out);

/*
 * desloc_step() for gradients that arrive in HOST memory (e.g. produced elsewhere and handed
 * over through pinned buffers): same step, with the host-to-device copies inside the call.
 *   host_grads : host array of M*num_tensors HOST pointers (page-locked memory if the copies
 *                are to overlap with compute), same indexing and dtype as for desloc_step().
 *   dev_grads  : host array of M*num_tensors DEVICE pointers to caller-owned staging buffers
 *                of the same sizes; they receive the copies and are what the kernels read.
 * The tensor list is cut into up to 8 groups; each group's gradients are copied on a stream
 * the context owns (tensors adjacent in both host and device memory go as one copy) and the
 * group's part of the step is launched on `stream` as soon as its copies have landed, so all
 * but the last group's compute hides behind the transfers.  The copies wait for work already
 * enqueued on `stream`.  Not available under stream capture (DESLOC_E_INVALID).
 */
DESLOC_API int desloc_step_host(desloc_ctx *ctx, int64_t t, float lr_t, float clip_bound_t,
                                const void *const *host_grads, void *const *dev_grads,
                                void *stream, uint32_t *mask_out);

/* As desloc_step() but with the sync mask given by the caller instead of derived from t
   (used to time or test one sync pattern in isolation).  mask bits outside X|U|V, or V for
   SGDM, are rejected with DESLOC_E_INVALID.  Counters are updated as for desloc_step(). */
DESLOC_API int desloc_step_masked(desloc_ctx *ctx, uint32_t mask, float lr_t, float clip_bound_t,
                       const void *const *grads, void *stream);

/*
 * One step with norm-based gradient clipping in front: worker m's whole gradient (all tensors)
 * is scaled by min(1, max_norm / ||g^m||_2) before the coordinate clip and the update.  This
 * is how the paper's language-model runs clipped (the model table of the experimental-details
 * appendix gives the bound on the gradient's L2 norm, 1.0, in its rho column); Algorithms 1-3
 * only have the coordinate-wise clip.  Costs one more read of the gradients: two reduction
 * launches (per-chunk partial sums in fp32, per-worker totals in fp64, fixed order, no
 * atomics) ahead of the step kernel, all enqueued on `stream` without host synchronisation.
 * max_norm must be > 0 and finite.  Other arguments as desloc_step().
 */
DESLOC_API int desloc_step_normclip(desloc_ctx *ctx, int64_t t, float lr_t, float clip_bound_t,
                                    float max_norm, const void *const *grads, void *stream,
                                    uint32_t *mask_out);

/*
 * Gradient norms ||g^m||_2 and clip factors of the latest desloc_step_normclip() into the host
 * arrays norms_out[M], scales_out[M] (either may be NULL).  Copies on `stream` and waits for
 * it: this call synchronises.
 */
DESLOC_API int desloc_get_grad_norms(desloc_ctx *ctx, float *norms_out, float *scales_out,
                                     void *stream);

/*
 * One step that also measures, per worker and per tensor, the L2 norms of
 *   kind 0: the gradient g_t^m as read (before any clipping),
 *   kind 1: the new parameters x_{t+1}^m as stored,
 *   kind 2: the update d_t^m of Algorithms 2-3 (eta_t u_t / sqrt(v_t + lambda^2) for Adam,
 *           eta_t u_t for ADOPT and SGDM; the weight-decay term is not part of it)
 * -- the gradient, parameter and update norms the paper tracks (gradient norms after the
 * workers are doubled, Section 6, RQ3; update and parameter norms of the billion-scale runs,
 * additional-results appendix).  The step kernel already has all three on chip, so the
 * sums of squares are formed there, one partial per (kind, worker, chunk): no extra pass over
 * memory, and the step computes exactly what desloc_step() computes.
 *   max_norm : > 0 puts norm-based clipping in front as desloc_step_normclip() does; 0 = off.
 * Other arguments as desloc_step().  Not available with desloc_step_host().
 */
DESLOC_API int desloc_step_diag(desloc_ctx *ctx, int64_t t, float lr_t, float clip_bound_t,
                                float max_norm, const void *const *grads, void *stream,
                                uint32_t *mask_out);

/*
 * Norms of the latest desloc_step_diag():
 *   per_tensor_out : host, [3][M][num_tensors] floats, entry (kind * M + m) * num_tensors + k,
 *                    or NULL;
 *   total_out      : host, [3][M] floats, the norm over the whole tensor list, or NULL.
 * Per-chunk partials are fp32; they are added per tensor, and the tensors per worker, in fp64
 * in a fixed order (no atomics: the same buffers and inputs give the same bits; where the chunks
 * of a tensor begin follows the alignment of worker 0's x, see desloc_plan_chunks_at()).  Two small launches on `stream`, then the
 * copies; the call waits for `stream`.  DESLOC_E_INVALID if no diagnostics step has run since
 * the context was created or its workers were changed.
 */
DESLOC_API int desloc_get_diag_norms(desloc_ctx *ctx, float *per_tensor_out, float *total_out,
                                     void *stream);

/*
 * Relative change of a state since a snapshot, per worker: out[m] = ||s^m - then^m||_2 /
 * ||then^m||_2 over the whole tensor list (the rate-of-change measure of Section 5.1,
 * "Metrics", ||s_{t+K} - s_t|| / ||s_t||).  array: 0 = x, 1 = u, 2 = v.  then: host array of
 * M*num_tensors DEVICE pointers to the caller's fp32 snapshot (same shapes as the state).
 * out: host array [M].  Enqueues on `stream` and waits for it: this call synchronises.
 */
DESLOC_API int desloc_rel_change(desloc_ctx *ctx, int32_t array, const float *const *then,
                                 float *out, void *stream);

/*
 * Change the set of workers between steps: add workers that start from the synchronised
 * state, or drop some (the paper's robustness claim: because every state is eventually
 * averaged, workers can join or leave; its experiment doubles the worker count mid-run,
 * Section 6, RQ3).
 *   M_new     : new worker count, 1..DESLOC_MAX_M.
 *   x, u, v   : host arrays of M_new*num_tensors DEVICE pointers, indexed as in desloc_create().
 *   first_new : workers 0..first_new-1 are taken as they are (normally the buffers of the
 *               workers that stay; their contents are not touched).  Workers first_new..M_new-1
 *               are new: every element of their x, u, v is overwritten with the mean over ALL
 *               workers the context held before the call (fp64 sum in worker order).
 *               first_new = M_new adds nobody (pure removal / re-ordering).
 * This call allocates (the pointer tables are re-made for the new count), waits for `stream`
 * before and after, and resets nothing else: counters and the step count continue.
 */
DESLOC_API int desloc_set_workers(desloc_ctx *ctx, int32_t M_new, int32_t first_new,
                                  float *const *x, float *const *u, float *const *v, void *stream);

/* Release the context and everything it allocated.  The caller's tensors are untouched.
   NULL is a no-op returning DESLOC_OK. */
DESLOC_API int desloc_destroy(desloc_ctx *ctx);

/* out[0..3] = steps taken, x-syncs, u-syncs, v-syncs (the per-array communication counts a
   distributed run of the same schedule would pay; Section 5.1 "Metrics"). */
DESLOC_API int desloc_get_counters(const desloc_ctx *ctx, int64_t out[4]);

/* Kernels launched by this context so far (one per step on the main path). */
DESLOC_API int64_t desloc_get_launch_count(const desloc_ctx *ctx);

/*
 * Multi-tensor plan: how the tensor list is cut into the chunks that thread blocks work
 * through.  Host-only.  Writes up to `cap` chunks as triples (tensor index, first element,
 * element count) into `out` (3*cap int64) and returns the total number of chunks the list
 * needs (which may exceed cap), or a negative desloc_status.
 * Every tensor starts a new chunk; chunks of a tensor are `chunk_elems` long except the last --
 * and except the first, where x0 says so:
 *   x0 : host array of num_tensors addresses, worker 0's x tensors (never dereferenced), or NULL.
 *        The copy engine is fastest on pieces that start on a 2 KB boundary, and needs 16-byte
 *        alignment at all.  So a tensor that does not start on a 2 KB boundary has its first
 *        chunk cut to the elements in front of the next one, and every later chunk starts on
 *        it -- for x and for every array laid out like x (the same element offsets in a
 *        buffer of its own).  A gradient laid out differently may end up 8 or 2 bytes off a
 *        16-byte boundary after the cut; such chunks are updated straight from global memory
 *        (128-bit accesses, or coordinate by coordinate), correctly but more slowly.
 * desloc_plan_chunks_at() with the x pointers given to desloc_create() is the table that context
 * works from; desloc_plan_chunks() is the same with x0 = NULL.
 */
DESLOC_API int64_t desloc_plan_chunks_at(const int64_t *numel, int32_t num_tensors, int64_t chunk_elems,
                                         const void *const *x0, int64_t *out, int64_t cap);
DESLOC_API int64_t desloc_plan_chunks(const int64_t *numel, int32_t num_tensors, int64_t chunk_elems,
                                      int64_t *out, int64_t cap);

/* Elements per chunk -- the run of tiles one thread block streams through, for all workers -- of
   a context created from cfg (M, numel and num_tensors are read).  A tile is 1024 elements for
   M <= 2, 512 for M = 3..8 (M > 8: 1024-element chunks, no tiles); a chunk is up to 8 tiles
   on a large problem, fewer on a small one.  Negative desloc_status on bad
   input. */
DESLOC_API int64_t desloc_chunk_elems(const desloc_config *cfg);

/*
 * desloc_step_static(): one step for callers that cannot allocate.  (The paper has no
 * counterpart; this is an interface variant, the update computed is desloc_step()'s.)
 *
 * desloc_create() takes device memory for its chunk and pointer tables.  That is not possible
 * for every caller: a process whose training framework has already claimed all of HBM for its
 * own memory pool gets an out-of-memory error from any further cudaMalloc (or forces the pool
 * to give memory back), and a latency-critical loop cannot afford the device-wide
 * synchronisation that cudaMalloc and cudaFree bring.  This entry point needs no context and
 * calls no cudaMalloc, cudaFree, cudaMallocHost or any other allocating routine: its tables
 * go into a fixed array inside the library image, DESLOC_STATIC_SCRATCH_BYTES (576 KB) of
 * device memory per GPU, held until the process exits.
 *
 * Limits: M * num_tensors <= DESLOC_STATIC_MAX_POINTERS, M <= 8, and at most
 * DESLOC_STATIC_MAX_CHUNKS chunks of desloc_chunk_elems(cfg) elements (every tensor starts a
 * new chunk) -- about 130 Mi parameters when tensors are large.  Anything bigger returns
 * DESLOC_E_TOO_LARGE and does nothing.
 *
 * Arguments as for desloc_create() + desloc_step(): cfg, the host arrays x, u, v, grads of
 * M*num_tensors DEVICE pointers (v may be NULL for SGDM), the step t, eta_t, the ADOPT bound,
 * the device and the stream.  State is updated in place; there are no counters.  All argument
 * checks happen before the first CUDA call, so a rejected call (NULL, range, invalid, too
 * large) touches neither the device nor the array.
 *
 * Set-up.  The first call on each device looks up the device address of the array
 * (cudaGetSymbolAddress, with that device current).  With the CUDA runtime's lazy module
 * loading that look-up is also the moment the runtime loads the module and reserves the
 * array's 576 KB on that GPU: make the first call at start-up -- before a framework's pool has
 * grown to fill the device, where it could fail with DESLOC_E_CUDA, and before any stream
 * capture begins.  The address is remembered per device for the life of the process and does
 * not survive a cudaDeviceReset().
 *
 * Uploads.  The library keeps a host copy of what it last wrote into the array.  A call
 * uploads only the tables that differ from it (the chunk table depends on the tensor list and
 * the alignment of worker 0's x, the four pointer tables on x, u, v, grads), from ordinary
 * pageable host memory, ahead of the kernel on `stream`; such a copy may wait for work already enqueued on `stream`
 * before it returns.  A loop that steps the same buffers every time uploads nothing after its
 * first call and only enqueues the kernel.  Because those copies read host memory the library
 * reuses, the call returns DESLOC_E_INVALID, enqueueing nothing, while `stream` is being
 * captured.
 *
 * Sharing.  All calls on a device share the one array, and it keeps the previous call's
 * tables: each call rewrites what it needs, nothing in it has to start at zero.  Host threads
 * are serialised inside the call, but two calls whose GPU work can overlap -- different
 * streams without an ordering between them -- race on the array and must be ordered by the
 * caller; calls issued one after the other on the same stream are safe.
 */
#define DESLOC_STATIC_MAX_POINTERS 2048
#define DESLOC_STATIC_MAX_CHUNKS 32768
#define DESLOC_STATIC_SCRATCH_BYTES (DESLOC_STATIC_MAX_CHUNKS * 16 + 4 * DESLOC_STATIC_MAX_POINTERS * 8)
DESLOC_API int desloc_step_static(const desloc_config *cfg, float *const *x, float *const *u,
                                  float *const *v, const void *const *grads, int64_t t,
                                  float lr_t, float clip_bound_t, int cuda_device, void *stream,
                                  uint32_t *mask_out);

/* Static description of a status code; never NULL. */
DESLOC_API const char *desloc_strerror(int status);

/* The last CUDA error code (cudaError_t as int) seen by this context, 0 if none. */
DESLOC_API int desloc_last_cuda_error(const desloc_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* DESLOC_H_ */
