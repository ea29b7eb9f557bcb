// Host-side pieces shared by the context path (desloc_host.cu) and the allocation-free entry
// point (desloc_static.cu): argument validation, the sync schedule, the chunk-size rule and the
// kernel-argument block, so that both paths validate, plan and launch identically.
#pragma once
#include <cmath>
#include <cstdint>
#include <limits>

#include <nvtx3/nvToolsExt.h>

#include "../../include/desloc.h"
#include "desloc_kernels.cuh"

namespace desloc {

// Polls a block gives its tile's copies before it gives up (each poll itself waits a while in
// hardware): far beyond any healthy latency, still finite.
constexpr int DEFAULT_WAIT_LIMIT = 1 << 22;

// A named range around every step call, visible to tools that record NVTX (no cost otherwise).
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
    NvtxRange(const NvtxRange &) = delete;
    NvtxRange &operator=(const NvtxRange &) = delete;
};

inline bool finite_in(float v, float lo, bool lo_incl, float hi, bool hi_incl) {
    if (!std::isfinite(v)) return false;
    if (lo_incl ? v < lo : v <= lo) return false;
    if (hi_incl ? v > hi : v >= hi) return false;
    return true;
}

// Everything about a desloc_config that can be checked without looking at numel or the device.
inline int validate_config(const desloc_config *c) {
    if (!c) return DESLOC_E_NULL;
    if (c->opt != DESLOC_ADAM && c->opt != DESLOC_ADOPT && c->opt != DESLOC_SGDM) return DESLOC_E_INVALID;
    if (c->grad_dtype != DESLOC_F32 && c->grad_dtype != DESLOC_BF16) return DESLOC_E_INVALID;
    if (c->flags & ~(DESLOC_FLAG_ADOPT_NORM_CLIP | DESLOC_FLAG_POST_AVERAGE)) return DESLOC_E_INVALID;
    if ((c->flags & DESLOC_FLAG_ADOPT_NORM_CLIP) && c->opt != DESLOC_ADOPT) return DESLOC_E_INVALID;
    if (c->M < 1 || c->M > DESLOC_MAX_M) return DESLOC_E_RANGE;
    if (c->num_tensors < 1) return DESLOC_E_RANGE;
    if (c->Kx < 0 || c->Ku < 0 || c->Kv < 0) return DESLOC_E_RANGE;
    if (!finite_in(c->beta1, 0.f, true, 1.f, false)) return DESLOC_E_RANGE;
    if (c->opt != DESLOC_SGDM && !finite_in(c->beta2, 0.f, true, 1.f, false)) return DESLOC_E_RANGE;
    if (!finite_in(c->eps, 0.f, true, std::numeric_limits<float>::max(), true)) return DESLOC_E_RANGE;
    if (!finite_in(c->weight_decay, 0.f, true, std::numeric_limits<float>::max(), true)) return DESLOC_E_RANGE;
    if (std::isnan(c->clip_rho)) return DESLOC_E_RANGE;
    return DESLOC_OK;
}

// numel[k] >= 1 for every tensor and a total that cannot overflow the byte arithmetic.
inline int validate_numel(const desloc_config *c, int64_t *total_out) {
    if (!c->numel) return DESLOC_E_NULL;
    int64_t total = 0;
    for (int32_t k = 0; k < c->num_tensors; ++k) {
        if (c->numel[k] < 1) return DESLOC_E_RANGE;
        if (c->numel[k] > (INT64_MAX >> 4) - total) return DESLOC_E_RANGE;
        total += c->numel[k];
    }
    if (total_out) *total_out = total;
    return DESLOC_OK;
}

// Per-step scalar arguments.
inline int validate_step(const desloc_config *c, float lr_t, float clip_bound_t) {
    if (!std::isfinite(lr_t)) return DESLOC_E_RANGE;
    if ((c->flags & DESLOC_FLAG_ADOPT_NORM_CLIP) && !(clip_bound_t >= 0.f)) return DESLOC_E_RANGE;
    return DESLOC_OK;
}

// Algorithm 1's three "t mod K = 0" tests, t from 0; K = 0 never syncs; SGDM has no second state.
inline uint32_t mask_at(const desloc_config *c, int64_t t) {
    uint32_t m = 0;
    if (c->Kx > 0 && t % c->Kx == 0) m |= DESLOC_SYNC_X;
    if (c->Ku > 0 && t % c->Ku == 0) m |= DESLOC_SYNC_U;
    if (c->opt != DESLOC_SGDM && c->Kv > 0 && t % c->Kv == 0) m |= DESLOC_SYNC_V;
    return m;
}

// Chunk length of a context: a run of tiles of the kernel that serves its worker count -- as
// many as amortise the per-chunk pointer look-up on a large problem (max_tiles_per_chunk), fewer
// on a small one, so that it still spreads over about four blocks per SM of a B200.
inline int64_t chunk_elems_for(int32_t M, const int64_t *numel, int32_t num_tensors) {
    const int64_t T = M <= MAX_MT ? tile_elems(M) : GENERIC_CHUNK_ELEMS;
    const int64_t most = M <= MAX_MT ? max_tiles_per_chunk(M) : 8;
    int64_t tiles = 0;
    for (int32_t k = 0; k < num_tensors; ++k) tiles += (numel[k] + T - 1) / T;
    int64_t per_chunk = tiles / (4 * 148);
    if (per_chunk < 1) per_chunk = 1;
    if (per_chunk > most) per_chunk = most;
    return per_chunk * T;
}

// Where the copy engine's 2 KB pieces start matters: measured on B200, tiles that begin 256 or
// 512 bytes off a 2 KB boundary of the fp32 arrays run 3 % slower than tiles on the boundary
// (1 KB off: 0.7 %).  So the first chunk of a tensor is cut short by `head` elements, such that
// every later chunk of it starts on a 2 KB boundary of worker 0's x -- and with it of every
// array that shares x's element offsets, the usual layout (one flat buffer per worker and array).
// The same cut turns a tensor that starts at an odd offset of a tightly packed buffer (x not
// 16-byte aligned: every chunk of it would take the scalar path), or at an odd multiple of four
// elements of a buffer padded to 16 bytes (x aligned, a bf16 gradient with the same offsets
// 8 bytes off), into a short head and an aligned rest.  A gradient that does NOT share x's
// offsets can lose its 16-byte alignment by the cut; where it keeps 8 bytes, the chunk is
// updated with 128-bit accesses from global memory (0.66-0.86 of the copy bandwidth), else
// coordinate by coordinate.
constexpr int64_t ALIGN_PHASE_ELEMS = 512;
inline int64_t head_elems(const void *x0, int64_t numel) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(x0);
    if ((a & 3u) != 0) return 0;
    const int64_t phase = static_cast<int64_t>(a >> 2) & (ALIGN_PHASE_ELEMS - 1);
    const int64_t head = (ALIGN_PHASE_ELEMS - phase) & (ALIGN_PHASE_ELEMS - 1);
    return head < numel ? head : 0;
}

// Chunks of one tensor: an optional short first chunk of `head` elements, then chunk_elems each.
inline int64_t chunks_of(int64_t numel, int64_t chunk_elems, int64_t head) {
    return (head > 0 ? 1 : 0) + (numel - head + chunk_elems - 1) / chunk_elems;
}

// heads: per tensor, elements of the short first chunk (0 = none), or nullptr for none at all.
inline int64_t count_chunks(const int64_t *numel, int32_t num_tensors, int64_t chunk_elems,
                            const int64_t *heads = nullptr) {
    int64_t n = 0;
    for (int32_t k = 0; k < num_tensors; ++k) n += chunks_of(numel[k], chunk_elems, heads ? heads[k] : 0);
    return n;
}

// One thread block per chunk (per worker and chunk where workers are separate work items): does
// the grid of a context with M workers fit, whatever the first chunks are cut to?
inline bool grid_fits(int32_t M, const int64_t *numel, int32_t num_tensors) {
    const int64_t nchunks = count_chunks(numel, num_tensors, chunk_elems_for(M, numel, num_tensors)) + num_tensors;
    const int64_t per_chunk = (M == 1 || M > MAX_MT) ? M : 1;
    return nchunks <= 0x7fffffffLL / per_chunk;
}

// Writes the chunk table for the list (every tensor starts a new chunk); `out` has room for
// count_chunks() entries.
inline void fill_chunks(const int64_t *numel, int32_t num_tensors, int64_t chunk_elems, Chunk *out,
                        const int64_t *heads = nullptr) {
    int64_t c = 0;
    for (int32_t k = 0; k < num_tensors; ++k) {
        const int64_t head = heads ? heads[k] : 0;
        if (head > 0) {
            out[c].tensor = k;
            out[c].count = static_cast<int32_t>(head);
            out[c].start = 0;
            ++c;
        }
        for (int64_t s = head; s < numel[k]; s += chunk_elems) {
            const int64_t left = numel[k] - s;
            out[c].tensor = k;
            out[c].count = static_cast<int32_t>(left < chunk_elems ? left : chunk_elems);
            out[c].start = s;
            ++c;
        }
    }
}

// The hyper-parameter part of the kernel arguments (tables and sizes are the caller's).
inline void fill_hyper(StepArgs &a, const desloc_config &c, float lr_t, float clip_bound_t) {
    a.nt = c.num_tensors;
    a.M = c.M;
    a.b1 = c.beta1;
    a.omb1 = static_cast<float>(1.0 - static_cast<double>(c.beta1));
    a.b2 = c.beta2;
    a.omb2 = static_cast<float>(1.0 - static_cast<double>(c.beta2));
    a.eps2 = static_cast<float>(static_cast<double>(c.eps) * static_cast<double>(c.eps));
    a.lam2 = static_cast<float>(static_cast<double>(c.eps) * static_cast<double>(c.eps));
    a.lr = lr_t;
    a.lrwd = static_cast<float>(static_cast<double>(lr_t) * static_cast<double>(c.weight_decay));
    a.rho = c.clip_rho > 0.f ? c.clip_rho : std::numeric_limits<float>::infinity();
    a.cbound = (c.flags & DESLOC_FLAG_ADOPT_NORM_CLIP) ? clip_bound_t
                                                       : std::numeric_limits<float>::infinity();
    a.wait_limit = DEFAULT_WAIT_LIMIT;
    a.err = nullptr;
    a.direct = 0;
}

// Which kernel a step of this configuration runs, and over how many blocks.
struct LaunchPlan {
    const void *fn = nullptr;
    long long grid = 0;
    bool strides = true;  // a smaller grid may stride over the work items (not the runtime-M kernel)
    int smem = 0;         // dynamic shared memory of the launch
    bool direct = false;  // too small to gain from staging: update straight from global memory
};

// Launches of at most this many blocks of single-tile chunks (two per SM of a B200: one wave)
// skip the staging.  Measured on the 4096-parameter, two-worker workload: 3.08 us per step in a
// CUDA graph of 16 steps against 3.34 us staged.
constexpr long long DIRECT_GRID = 2 * 148;

// The tile kernels use more than the 48 KB of shared memory a kernel gets by default: raise the
// function's limit to what the launch asks for.  Not an allocation.
inline cudaError_t prepare_launch(const LaunchPlan &p) {
    if (p.smem <= 32 * 1024) return cudaSuccess;   // with the kernel's static part still under 48 KB
    return cudaFuncSetAttribute(p.fn, cudaFuncAttributeMaxDynamicSharedMemorySize, p.smem);
}

inline LaunchPlan plan_launch(const desloc_config &c, uint32_t mask, long long nchunks, bool diag) {
    LaunchPlan p;
    // The mean of one replica is the replica: M = 1 always runs the local kernel.
    const uint32_t kmask = (c.M == 1) ? 0u : mask;
    const bool post = (c.flags & DESLOC_FLAG_POST_AVERAGE) != 0;
    const bool bf16 = c.grad_dtype == DESLOC_BF16;
    const bool per_worker_items = (c.M == 1) || (kmask == 0 && c.M > MAX_MT);
    const bool generic = kmask != 0 && c.M > MAX_MT;
    p.fn = generic ? lookup_generic_kernel(c.opt, post, bf16, static_cast<int>(kmask), diag)
                   : lookup_step_kernel(c.opt, post, bf16, c.M, static_cast<int>(kmask), diag);
    p.strides = !generic;
    p.smem = generic ? 0 : step_smem_bytes(c.opt, per_worker_items ? 1 : c.M, bf16);
    p.grid = per_worker_items ? nchunks * c.M : nchunks;
    const int mt = per_worker_items ? 1 : c.M;
    p.direct = p.grid <= DIRECT_GRID && mt <= MAX_MT &&
               chunk_elems_for(c.M, c.numel, c.num_tensors) == tile_elems(mt);
    return p;
}

}  // namespace desloc
