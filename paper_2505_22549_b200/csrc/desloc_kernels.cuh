// DES-LOC fused step kernel for sm_100a: one streaming pass over g, x, u, v of all M
// worker replicas (Algorithm 1 with the Adam, ADOPT and SGDM rules of Algorithms 2-3).
//
// Work decomposition.  The tensor list is cut into chunks of CHUNK_ELEMS elements of one
// tensor (table built once on the host).  A thread block takes one chunk at a time:
//   * for M = 2..8 the kernel is instantiated per worker count MT = M and per sync mask
//     (mask 0 = local step): a thread loads its elements of all M replicas, sums the synced
//     arrays in a fixed tree order, and writes every replica back -- a sync step moves the
//     same bytes as a local step, through the same code shape;
//   * desloc_local_kernel serves M = 1 and local steps of M > 8: workers are independent
//     there, so the work item is (worker, group of four consecutive chunks).
// Every thread issues all loads of a batch (up to four workers x 4 arrays, 128-bit where
// aligned) before the first use, so that enough bytes are in flight to cover HBM latency;
// the arithmetic is fp32.  Tensors whose pointers are not 16-byte aligned and the last
// (numel mod 4) elements of a tensor take the scalar instantiation of the same code.
//
// Measured choices (B200; fractions are of the device's copy bandwidth):
//   * plain loads and stores: evict-first (.cs) accesses were 2 % slower on every workload;
//   * IEEE sqrt and division: the hardware reciprocal square root was not faster here;
//   * 256 threads, three resident blocks per SM for M <= 4 (two or four: 9-10 % slower);
//   * more than four workers: means first, then the workers in balanced batches that fit the
//     register budget of three blocks per SM (0.96-0.99 against 0.89-0.95 all at once).
//
// DIAG instantiations also accumulate, from values already in registers, the squared L2 norms
// of the gradient as read, of the update d_t and of the new parameters per (worker, chunk):
// no extra pass over memory, 12 bytes written per worker and chunk.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace desloc {

constexpr int OPT_ADAM = 0, OPT_ADOPT = 1, OPT_SGDM = 2;
constexpr int SYNC_X = 1, SYNC_U = 2, SYNC_V = 4;
constexpr int BLOCK_THREADS = 256;
constexpr int CHUNK_ELEMS = BLOCK_THREADS * 16;  // 256 threads x 4 elements x 4 rounds = 4096
constexpr int MAX_MT = 8;          // largest worker count with a register-resident kernel
constexpr int DIAG_G = 0, DIAG_X = 1, DIAG_D = 2, DIAG_KINDS = 3;

struct __align__(16) Chunk {
    int32_t tensor;  // index into the tensor list
    int32_t count;   // elements in this chunk (<= CHUNK_ELEMS)
    int64_t start;   // first element within the tensor
};

constexpr int INLINE_PTRS = 32;  // gradient pointers that fit in the kernel parameters

struct StepArgs {
    const Chunk *chunks;
    long long nchunks;
    float *const *x;  // device tables [M * nt], entry m * nt + k
    float *const *u;
    float *const *v;
    const void *const *g;                // device table, or nullptr: use g_inline
    const void *g_inline[INLINE_PTRS];   // small problems under stream capture (no table upload)
    const float *gscale;  // per-worker factor applied to g before the clip, or nullptr (= 1)
    float *diag;          // DIAG kernels: [DIAG_KINDS][M][diag_stride] partial sums of squares
    long long diag_stride;  // chunks of the whole context (a launch may cover a sub-range)
    long long diag_chunk0;  // index of chunks[0] within the context's chunk table
    int nt;
    int M;
    float b1, omb1;   // beta1, 1 - beta1
    float b2, omb2;   // beta2, 1 - beta2
    float eps;        // ADOPT epsilon
    float lam2;       // Adam lambda^2
    float lr;         // eta_t
    float lrwd;       // eta_t * weight_decay
    float rho;        // coordinate clip radius, +inf when off
    float cbound;     // ADOPT normalised-gradient bound, +inf when off
};

__device__ __forceinline__ const void *grad_ptr(const StepArgs &a, long long idx) {
    return a.g ? a.g[idx] : a.g_inline[idx];
}

struct bf16_t {
    uint16_t bits;
};

template <int VEC>
struct FV {
    float a[VEC];
};

// ---- global memory access: 128-bit or scalar ----------------------------------------------
template <int VEC>
__device__ __forceinline__ FV<VEC> ld_f32(const char *base, long long elem) {
    FV<VEC> r;
    if constexpr (VEC == 4) {
        const float4 t = *(reinterpret_cast<const float4 *>(base) + (elem >> 2));
        r.a[0] = t.x; r.a[1] = t.y; r.a[2] = t.z; r.a[3] = t.w;
    } else {
        r.a[0] = *(reinterpret_cast<const float *>(base) + elem);
    }
    return r;
}

template <int VEC>
__device__ __forceinline__ void st_f32(char *base, long long elem, const FV<VEC> &r) {
    if constexpr (VEC == 4) {
        *(reinterpret_cast<float4 *>(base) + (elem >> 2)) = make_float4(r.a[0], r.a[1], r.a[2], r.a[3]);
    } else {
        *(reinterpret_cast<float *>(base) + elem) = r.a[0];
    }
}

template <int VEC, typename GT>
__device__ __forceinline__ FV<VEC> ld_grad(const char *base, long long elem) {
    FV<VEC> r;
    if constexpr (sizeof(GT) == 4) {
        r = ld_f32<VEC>(base, elem);
    } else if constexpr (VEC == 4) {
        // four bf16 in 8 bytes; bf16 -> fp32 is a 16-bit shift (exact)
        const uint2 t = *(reinterpret_cast<const uint2 *>(base) + (elem >> 2));
        r.a[0] = __uint_as_float(t.x << 16);
        r.a[1] = __uint_as_float(t.x & 0xffff0000u);
        r.a[2] = __uint_as_float(t.y << 16);
        r.a[3] = __uint_as_float(t.y & 0xffff0000u);
    } else {
        const unsigned short t = *(reinterpret_cast<const unsigned short *>(base) + elem);
        r.a[0] = __uint_as_float(static_cast<unsigned>(t) << 16);
    }
    return r;
}

template <int VEC>
__device__ __forceinline__ float sum_sq(const FV<VEC> &r) {
    float s = r.a[0] * r.a[0];
#pragma unroll
    for (int c = 1; c < VEC; ++c) s = fmaf(r.a[c], r.a[c], s);
    return s;
}

// ---- diagnostics accumulator ----------------------------------------------------------------
// Per-thread running sums of squares in shared memory, slot [kind][worker slot][thread]: they
// outlive the rounds of a chunk without occupying registers.  flush() reduces them over the
// block (shuffle tree, then the warp sums in order: deterministic) and hands thread
// j < DIAG_KINDS * NW the total of slot j.
template <bool DIAG, int NW>
struct DiagAcc {
    float *slots;  // [DIAG_KINDS * NW][BLOCK_THREADS]
    float *wsum;   // [DIAG_KINDS * NW][BLOCK_THREADS / 32]
    int base;      // added to the worker slot (the ragged path of the local kernel)

    __device__ __forceinline__ void clear() const {
        if constexpr (DIAG) {
#pragma unroll
            for (int j = 0; j < DIAG_KINDS * NW; ++j) slots[j * BLOCK_THREADS + threadIdx.x] = 0.f;
        }
    }
    __device__ __forceinline__ void add(int kind, int m, float v) const {
        if constexpr (DIAG) slots[(kind * NW + base + m) * BLOCK_THREADS + threadIdx.x] += v;
    }
    // All threads call; returns slot `threadIdx.x`'s block total in threads < DIAG_KINDS * NW
    // and zeroes the slots.  Contains a block barrier.
    __device__ __forceinline__ float flush() const {
        float total = 0.f;
        if constexpr (DIAG) {
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
            for (int j = 0; j < DIAG_KINDS * NW; ++j) {
                float v = slots[j * BLOCK_THREADS + threadIdx.x];
                slots[j * BLOCK_THREADS + threadIdx.x] = 0.f;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
                if (lane == 0) wsum[j * (BLOCK_THREADS / 32) + warp] = v;
            }
            __syncthreads();
            if (threadIdx.x < DIAG_KINDS * NW) {
#pragma unroll
                for (int w = 0; w < BLOCK_THREADS / 32; ++w)
                    total += wsum[threadIdx.x * (BLOCK_THREADS / 32) + w];
            }
        }
        return total;
    }
};

// ---- the update of one coordinate across all MT workers (registers only) -----------------
// Pre-average (Algorithms 1-3): synced arrays are replaced by their worker mean BEFORE the
// update.  Post-average (Algorithms 4-5): the updated values are averaged, and the parameter
// step uses the averaged states.
// Worker sum as a fixed binary tree: the first 2^k workers (2^k the largest power of two
// below the count) against the rest, recursively -- ((s0+s1)+(s2+s3))+((s4+s5)+(s6+s7)) for
// eight.  Deterministic, and exact when all M values are equal and M is a power of two.
template <int LO, int N, int MT>
__device__ __forceinline__ float tree_sum(const float (&s)[MT]) {
    if constexpr (N == 1) {
        return s[LO];
    } else {
        constexpr int H = (N > 4) ? 4 : (N > 2 ? 2 : 1);
        static_assert(N <= 8, "tree_sum covers up to eight workers");
        return tree_sum<LO, H, MT>(s) + tree_sum<LO + H, N - H, MT>(s);
    }
}

template <int MT>
__device__ __forceinline__ float mean_of(const float (&s)[MT]) {
    return tree_sum<0, MT, MT>(s) / static_cast<float>(MT);
}

// One worker's state update from the clipped gradient: `up`, `vp` are the previous states the
// update starts from (the worker's own or the worker mean); `vown` is always the worker's own
// previous v, which ADOPT's normaliser uses (Algorithm 3).
// FAST: hardware reciprocal square root (2 ulp) in place of IEEE sqrt and division.  Only the
// runtime-M kernel uses it: that kernel is bound by instruction issue, not by memory, and the
// exact forms cost it a tenth of its speed.
template <int OPT, bool FAST = false>
__device__ __forceinline__ void state_update(const StepArgs &a, float g, float up, float vp,
                                             float vown, float &un, float &vn) {
    // coordinate-wise clip: sgn(g) min(|g|, rho)  (Section 3.1); rho = +inf when off
    const float gh = fminf(fmaxf(g, -a.rho), a.rho);
    if constexpr (OPT == OPT_ADAM) {
        un = fmaf(a.b1, up, a.omb1 * gh);
        vn = fmaf(a.b2, vp, (a.omb2 * gh) * gh);
    } else if constexpr (OPT == OPT_ADOPT) {
        vn = fmaf(a.b2, vp, (a.omb2 * gh) * gh);
        float r;
        if constexpr (FAST)
            r = gh * rsqrtf(fmaxf(vown, a.eps * a.eps));  // 1 / max(sqrt(v), eps)
        else
            r = gh / fmaxf(sqrtf(vown), a.eps);
        r = fminf(fmaxf(r, -a.cbound), a.cbound);
        un = fmaf(a.b1, up, a.omb1 * r);
    } else {
        un = fmaf(a.b1, up, a.omb1 * gh);
        vn = 0.f;
    }
}

// The update d_t of Algorithms 2-3 from the new states.
template <int OPT, bool FAST = false>
__device__ __forceinline__ float direction(const StepArgs &a, float un, float vn) {
    if constexpr (OPT == OPT_ADAM)
        return FAST ? (a.lr * un) * rsqrtf(vn + a.lam2) : (a.lr * un) / sqrtf(vn + a.lam2);
    else
        return a.lr * un;
}

// x* (1 - eta wd) - d, written as x* - (eta wd x* + d): one rounding at x's scale
__device__ __forceinline__ float apply_step(const StepArgs &a, float xp, float d) {
    return xp - fmaf(a.lrwd, xp, d);
}

// All MT workers of one coordinate at once.  On return x, u, v hold the new values and d the
// update each worker applied.
template <int OPT, int MASK, int MT, bool POST>
__device__ __forceinline__ void update_coord(const StepArgs &a, const float (&g)[MT],
                                             float (&x)[MT], float (&u)[MT], float (&v)[MT],
                                             float (&d)[MT]) {
    constexpr bool PRE = !POST;
    float xb = 0.f, ub = 0.f, vb = 0.f;
    if constexpr (PRE && (MASK & SYNC_X)) xb = mean_of<MT>(x);
    if constexpr (PRE && (MASK & SYNC_U)) ub = mean_of<MT>(u);
    if constexpr (PRE && (MASK & SYNC_V) && OPT != OPT_SGDM) vb = mean_of<MT>(v);

    float un[MT], vn[MT], xn[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        const float up = (PRE && (MASK & SYNC_U)) ? ub : u[m];
        const float vp = (PRE && (MASK & SYNC_V)) ? vb : v[m];
        state_update<OPT>(a, g[m], up, vp, v[m], un[m], vn[m]);
    }
    if constexpr (POST && (MASK & SYNC_U)) {
        const float mu = mean_of<MT>(un);
#pragma unroll
        for (int m = 0; m < MT; ++m) un[m] = mu;
    }
    if constexpr (POST && (MASK & SYNC_V) && OPT != OPT_SGDM) {
        const float mv = mean_of<MT>(vn);
#pragma unroll
        for (int m = 0; m < MT; ++m) vn[m] = mv;
    }
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        const float xp = (PRE && (MASK & SYNC_X)) ? xb : x[m];
        d[m] = direction<OPT>(a, un[m], vn[m]);
        xn[m] = apply_step(a, xp, d[m]);
    }
    if constexpr (POST && (MASK & SYNC_X)) {
        const float mx = mean_of<MT>(xn);
#pragma unroll
        for (int m = 0; m < MT; ++m) xn[m] = mx;
    }
#pragma unroll
    for (int m = 0; m < MT; ++m) {
        x[m] = xn[m];
        u[m] = un[m];
        v[m] = vn[m];
    }
}

// ---- many workers (MT > 4): batches that fit the register budget --------------------------
// Registers a worker costs while its batch is in flight (FV<4> = 4 registers; bf16 g = 2).
template <int OPT, typename GT>
__host__ __device__ constexpr int worker_regs(bool ld_x, bool ld_u, bool ld_v) {
    return (sizeof(GT) == 2 ? 2 : 4) + 4 * ((ld_x ? 1 : 0) + (ld_u ? 1 : 0) + (ld_v ? 1 : 0));
}
// Largest batch within `budget` registers, then balanced over the batches needed
// (8 workers at up to 3 per batch run as 3 + 3 + 2).
__host__ __device__ constexpr int batch_size(int left, int per_worker, int budget) {
    int bmax = budget / per_worker;
    if (bmax < 1) bmax = 1;
    if (bmax > 4) bmax = 4;
    const int nb = (left + bmax - 1) / bmax;
    return (left + nb - 1) / nb;
}

template <int VEC, int MT>
__device__ __forceinline__ FV<VEC> mean_over_workers(char *const *bases, long long e) {
    FV<VEC> S[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) S[m] = ld_f32<VEC>(bases[m], e);
    FV<VEC> r;
#pragma unroll
    for (int c = 0; c < VEC; ++c) {
        float s[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) s[m] = S[m].a[c];
        r.a[c] = mean_of<MT>(s);
    }
    return r;
}

// Pre-average tile: the arrays to be averaged are loaded for all MT workers and reduced to
// their means; the per-worker phase then runs over batches, loading only what is not averaged
// (ADOPT also its own v).  Same loads, same arithmetic, same summation tree -- bitwise the
// same result as the all-at-once tile.
template <int OPT, int MASK, int MT, typename GT, int VEC, bool DIAG, int M0, int B, int NW>
__device__ __forceinline__ void pre_worker_batch(const StepArgs &a, char *const (*sp)[MT],
                                                 const float *sscale, long long e,
                                                 const FV<VEC> &xb, const FV<VEC> &ub,
                                                 const FV<VEC> &vb, const DiagAcc<DIAG, NW> &dg) {
    constexpr bool SX = MASK & SYNC_X, SU = MASK & SYNC_U;
    constexpr bool SV = (MASK & SYNC_V) && OPT != OPT_SGDM;
    constexpr bool NEED_V = OPT != OPT_SGDM && (!SV || OPT == OPT_ADOPT);
    FV<VEC> G[B], X[B], U[B], V[B];
#pragma unroll
    for (int b = 0; b < B; ++b) {
        G[b] = ld_grad<VEC, GT>(sp[3][M0 + b], e);
        if constexpr (!SX) X[b] = ld_f32<VEC>(sp[0][M0 + b], e);
        if constexpr (!SU) U[b] = ld_f32<VEC>(sp[1][M0 + b], e);
        if constexpr (NEED_V) V[b] = ld_f32<VEC>(sp[2][M0 + b], e);
    }
#pragma unroll
    for (int b = 0; b < B; ++b) {
        dg.add(DIAG_G, M0 + b, sum_sq<VEC>(G[b]));
        FV<VEC> D;
#pragma unroll
        for (int c = 0; c < VEC; ++c) {
            const float up = SU ? ub.a[c] : U[b].a[c];
            const float vown = NEED_V ? V[b].a[c] : 0.f;
            const float vp = SV ? vb.a[c] : vown;
            const float xp = SX ? xb.a[c] : X[b].a[c];
            float un, vn;
            state_update<OPT>(a, G[b].a[c] * sscale[M0 + b], up, vp, vown, un, vn);
            D.a[c] = direction<OPT>(a, un, vn);
            X[b].a[c] = apply_step(a, xp, D.a[c]);
            U[b].a[c] = un;
            V[b].a[c] = vn;
        }
        dg.add(DIAG_D, M0 + b, sum_sq<VEC>(D));
        dg.add(DIAG_X, M0 + b, sum_sq<VEC>(X[b]));
        st_f32<VEC>(sp[0][M0 + b], e, X[b]);
        st_f32<VEC>(sp[1][M0 + b], e, U[b]);
        if constexpr (OPT != OPT_SGDM) st_f32<VEC>(sp[2][M0 + b], e, V[b]);
    }
}

template <int OPT, int MASK, int MT, typename GT, int VEC, bool DIAG, int M0, int NW>
__device__ __forceinline__ void pre_worker_batches(const StepArgs &a, char *const (*sp)[MT],
                                                   const float *sscale, long long e,
                                                   const FV<VEC> &xb, const FV<VEC> &ub,
                                                   const FV<VEC> &vb, const DiagAcc<DIAG, NW> &dg) {
    if constexpr (M0 < MT) {
        constexpr bool SX = MASK & SYNC_X, SU = MASK & SYNC_U;
        constexpr bool SV = (MASK & SYNC_V) && OPT != OPT_SGDM;
        constexpr bool NEED_V = OPT != OPT_SGDM && (!SV || OPT == OPT_ADOPT);
        // 80 registers per thread at three blocks per SM; the means, addresses and constants
        // take about 28 of them
        constexpr int B = batch_size(MT - M0, worker_regs<OPT, GT>(!SX, !SU, NEED_V), 56);
        pre_worker_batch<OPT, MASK, MT, GT, VEC, DIAG, M0, B>(a, sp, sscale, e, xb, ub, vb, dg);
        pre_worker_batches<OPT, MASK, MT, GT, VEC, DIAG, M0 + B>(a, sp, sscale, e, xb, ub, vb, dg);
    }
}

template <int OPT, int MASK, int MT, typename GT, int VEC, bool DIAG, int NW>
__device__ __forceinline__ void process_tile_pre_batched(const StepArgs &a, char *const (*sp)[MT],
                                                         const float *sscale, long long e,
                                                         const DiagAcc<DIAG, NW> &dg) {
    FV<VEC> xb{}, ub{}, vb{};
    if constexpr (MASK & SYNC_X) xb = mean_over_workers<VEC, MT>(sp[0], e);
    if constexpr (MASK & SYNC_U) ub = mean_over_workers<VEC, MT>(sp[1], e);
    if constexpr ((MASK & SYNC_V) && OPT != OPT_SGDM) vb = mean_over_workers<VEC, MT>(sp[2], e);
    pre_worker_batches<OPT, MASK, MT, GT, VEC, DIAG, 0>(a, sp, sscale, e, xb, ub, vb, dg);
}

// Post-average tile for MT > 4.  Every worker stores the MEAN of a synced array, so only the
// running tree sums of the updated values have to survive a batch, not the values themselves:
// the sum tree of up to eight workers is (first four) + (the rest), which is exactly two
// batches.  Phase A updates the states batch by batch; an array that is not synced is stored
// at once.  The parameter step of a worker needs its final states: when those are all its own
// (no synced state enters d_t) it also runs in phase A; otherwise phase B loads x after the
// means are known.  Only when Adam syncs exactly one of u, v does phase B need the other one
// per worker: that one array is kept in registers.  Same arithmetic and summation tree as the
// all-at-once tile.
template <int OPT, int MASK>
struct PostPlan {
    static constexpr bool SX = MASK & SYNC_X, SU = MASK & SYNC_U;
    static constexpr bool SV = (MASK & SYNC_V) && OPT != OPT_SGDM;
    // does d_t depend on a state that is averaged?
    static constexpr bool D_NEEDS_MEAN = SU || (OPT == OPT_ADAM && SV);
    static constexpr bool KEEP_U = D_NEEDS_MEAN && !SU;                      // Adam, v synced only
    static constexpr bool KEEP_V = D_NEEDS_MEAN && OPT == OPT_ADAM && !SV;   // Adam, u synced only
};

template <int VEC, int B>
__device__ __forceinline__ FV<VEC> group_sum(const FV<VEC> (&S)[B]) {
    FV<VEC> r;
#pragma unroll
    for (int c = 0; c < VEC; ++c) {
        float s[B];
#pragma unroll
        for (int b = 0; b < B; ++b) s[b] = S[b].a[c];
        r.a[c] = tree_sum<0, B, B>(s);
    }
    return r;
}

template <int OPT, int MASK, int MT, typename GT, int VEC, bool DIAG, int M0, int B, int NW>
__device__ __forceinline__ void post_phase_a(const StepArgs &a, char *const (*sp)[MT],
                                             const float *sscale, long long e, FV<VEC> &su,
                                             FV<VEC> &sv, FV<VEC> &sx, FV<VEC> (&keep)[MT],
                                             const DiagAcc<DIAG, NW> &dg) {
    using P = PostPlan<OPT, MASK>;
    FV<VEC> G[B], U[B], V[B], X[B];
#pragma unroll
    for (int b = 0; b < B; ++b) {
        G[b] = ld_grad<VEC, GT>(sp[3][M0 + b], e);
        U[b] = ld_f32<VEC>(sp[1][M0 + b], e);
        if constexpr (OPT != OPT_SGDM) V[b] = ld_f32<VEC>(sp[2][M0 + b], e);
        if constexpr (!P::D_NEEDS_MEAN) X[b] = ld_f32<VEC>(sp[0][M0 + b], e);
    }
#pragma unroll
    for (int b = 0; b < B; ++b) {
        dg.add(DIAG_G, M0 + b, sum_sq<VEC>(G[b]));
        FV<VEC> D;
#pragma unroll
        for (int c = 0; c < VEC; ++c) {
            const float vown = OPT != OPT_SGDM ? V[b].a[c] : 0.f;
            float un, vn;
            state_update<OPT>(a, G[b].a[c] * sscale[M0 + b], U[b].a[c], vown, vown, un, vn);
            U[b].a[c] = un;
            V[b].a[c] = vn;
            if constexpr (!P::D_NEEDS_MEAN) {
                D.a[c] = direction<OPT>(a, un, vn);
                X[b].a[c] = apply_step(a, X[b].a[c], D.a[c]);
            }
        }
        if constexpr (!P::SU && !P::KEEP_U) st_f32<VEC>(sp[1][M0 + b], e, U[b]);
        if constexpr (OPT != OPT_SGDM && !P::SV && !P::KEEP_V) st_f32<VEC>(sp[2][M0 + b], e, V[b]);
        if constexpr (P::KEEP_U) keep[M0 + b] = U[b];
        if constexpr (P::KEEP_V) keep[M0 + b] = V[b];
        if constexpr (!P::D_NEEDS_MEAN) {
            dg.add(DIAG_D, M0 + b, sum_sq<VEC>(D));
            if constexpr (!P::SX) {
                dg.add(DIAG_X, M0 + b, sum_sq<VEC>(X[b]));
                st_f32<VEC>(sp[0][M0 + b], e, X[b]);
            }
        }
    }
    // this batch's node of the sum tree
    const bool first = M0 == 0;
    if constexpr (P::SU) {
        const FV<VEC> s = group_sum<VEC, B>(U);
#pragma unroll
        for (int c = 0; c < VEC; ++c) su.a[c] = first ? s.a[c] : su.a[c] + s.a[c];
    }
    if constexpr (P::SV) {
        const FV<VEC> s = group_sum<VEC, B>(V);
#pragma unroll
        for (int c = 0; c < VEC; ++c) sv.a[c] = first ? s.a[c] : sv.a[c] + s.a[c];
    }
    if constexpr (P::SX && !P::D_NEEDS_MEAN) {
        const FV<VEC> s = group_sum<VEC, B>(X);
#pragma unroll
        for (int c = 0; c < VEC; ++c) sx.a[c] = first ? s.a[c] : sx.a[c] + s.a[c];
    }
}

template <int OPT, int MASK, int MT, int VEC, bool DIAG, int M0, int B, int NW>
__device__ __forceinline__ void post_phase_b(const StepArgs &a, char *const (*sp)[MT], long long e,
                                             const FV<VEC> &mu, const FV<VEC> &mv, FV<VEC> &sx,
                                             const FV<VEC> (&keep)[MT],
                                             const DiagAcc<DIAG, NW> &dg) {
    using P = PostPlan<OPT, MASK>;
    FV<VEC> X[B];
#pragma unroll
    for (int b = 0; b < B; ++b) X[b] = ld_f32<VEC>(sp[0][M0 + b], e);
#pragma unroll
    for (int b = 0; b < B; ++b) {
        FV<VEC> D;
#pragma unroll
        for (int c = 0; c < VEC; ++c) {
            const float un = P::SU ? mu.a[c] : keep[M0 + b].a[c];
            const float vn = P::SV ? mv.a[c] : (P::KEEP_V ? keep[M0 + b].a[c] : 0.f);
            D.a[c] = direction<OPT>(a, un, vn);
            X[b].a[c] = apply_step(a, X[b].a[c], D.a[c]);
        }
        dg.add(DIAG_D, M0 + b, sum_sq<VEC>(D));
        if constexpr (!P::SX) {
            dg.add(DIAG_X, M0 + b, sum_sq<VEC>(X[b]));
            st_f32<VEC>(sp[0][M0 + b], e, X[b]);
        }
        if constexpr (P::SU) st_f32<VEC>(sp[1][M0 + b], e, mu);
        if constexpr (P::KEEP_U) st_f32<VEC>(sp[1][M0 + b], e, keep[M0 + b]);
        if constexpr (P::SV) st_f32<VEC>(sp[2][M0 + b], e, mv);
        if constexpr (P::KEEP_V) st_f32<VEC>(sp[2][M0 + b], e, keep[M0 + b]);
    }
    if constexpr (P::SX) {
        const FV<VEC> s = group_sum<VEC, B>(X);
#pragma unroll
        for (int c = 0; c < VEC; ++c) sx.a[c] = (M0 == 0) ? s.a[c] : sx.a[c] + s.a[c];
    }
}

template <int OPT, int MASK, int MT, typename GT, int VEC, bool DIAG, int NW>
__device__ __forceinline__ void process_tile_post_batched(const StepArgs &a, char *const (*sp)[MT],
                                                          const float *sscale, long long e,
                                                          const DiagAcc<DIAG, NW> &dg) {
    using P = PostPlan<OPT, MASK>;
    static_assert(MT > 4 && MT <= 8, "two batches: the first four workers and the rest");
    FV<VEC> su{}, sv{}, sx{};
    FV<VEC> keep[MT];  // only touched (and only then given registers) when Adam keeps one state
    post_phase_a<OPT, MASK, MT, GT, VEC, DIAG, 0, 4>(a, sp, sscale, e, su, sv, sx, keep, dg);
    post_phase_a<OPT, MASK, MT, GT, VEC, DIAG, 4, MT - 4>(a, sp, sscale, e, su, sv, sx, keep, dg);
    // the means divide the tree sum by MT, as mean_of does
#pragma unroll
    for (int c = 0; c < VEC; ++c) {
        if constexpr (P::SU) su.a[c] = su.a[c] / static_cast<float>(MT);
        if constexpr (P::SV) sv.a[c] = sv.a[c] / static_cast<float>(MT);
    }
    if constexpr (P::D_NEEDS_MEAN && !(P::KEEP_U || P::KEEP_V)) {
        // nothing is kept per worker: all MT loads of x go out together
        post_phase_b<OPT, MASK, MT, VEC, DIAG, 0, MT>(a, sp, e, su, sv, sx, keep, dg);
    } else if constexpr (P::D_NEEDS_MEAN) {
        post_phase_b<OPT, MASK, MT, VEC, DIAG, 0, 4>(a, sp, e, su, sv, sx, keep, dg);
        post_phase_b<OPT, MASK, MT, VEC, DIAG, 4, MT - 4>(a, sp, e, su, sv, sx, keep, dg);
    } else {
        // phase A already stepped x; the synced states still have to be written
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            if constexpr (P::SU) st_f32<VEC>(sp[1][m], e, su);
            if constexpr (P::SV) st_f32<VEC>(sp[2][m], e, sv);
        }
    }
    if constexpr (P::SX) {
#pragma unroll
        for (int c = 0; c < VEC; ++c) sx.a[c] = sx.a[c] / static_cast<float>(MT);
        const float xx = sum_sq<VEC>(sx);
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            dg.add(DIAG_X, m, xx);
            st_f32<VEC>(sp[0][m], e, sx);
        }
    }
}

// ---- one thread's tile: MT workers x VEC elements at position e ----------------------------
// sp[arr][m] are chunk-relative base pointers in shared memory (arr: 0 x, 1 u, 2 v, 3 g).
template <int OPT, int MASK, int MT, typename GT, bool POST, int VEC, bool DIAG, int NW>
__device__ __forceinline__ void process_tile(const StepArgs &a, char *const (*sp)[MT],
                                             const float *sscale, long long e,
                                             const DiagAcc<DIAG, NW> &dg) {
    if constexpr (MT > 4 && !POST && OPT != OPT_SGDM) {
        process_tile_pre_batched<OPT, MASK, MT, GT, VEC, DIAG>(a, sp, sscale, e, dg);
        return;
    } else if constexpr (MT > 4 && POST && MASK != 0 && OPT != OPT_SGDM) {
        process_tile_post_batched<OPT, MASK, MT, GT, VEC, DIAG>(a, sp, sscale, e, dg);
        return;
    } else {
        // all at once: M <= 4, and SGDM (one state less) for every M
        FV<VEC> G[MT], X[MT], U[MT], V[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            G[m] = ld_grad<VEC, GT>(sp[3][m], e);
            X[m] = ld_f32<VEC>(sp[0][m], e);
            U[m] = ld_f32<VEC>(sp[1][m], e);
            if constexpr (OPT != OPT_SGDM) V[m] = ld_f32<VEC>(sp[2][m], e);
        }
        if constexpr (DIAG) {
#pragma unroll
            for (int m = 0; m < MT; ++m) dg.add(DIAG_G, m, sum_sq<VEC>(G[m]));
        }
        float dd[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) dd[m] = 0.f;
#pragma unroll
        for (int c = 0; c < VEC; ++c) {
            float g[MT], x[MT], u[MT], v[MT], d[MT];
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                g[m] = G[m].a[c] * sscale[m];
                x[m] = X[m].a[c];
                u[m] = U[m].a[c];
                v[m] = (OPT != OPT_SGDM) ? V[m].a[c] : 0.f;
            }
            update_coord<OPT, MASK, MT, POST>(a, g, x, u, v, d);
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                X[m].a[c] = x[m];
                U[m].a[c] = u[m];
                if constexpr (OPT != OPT_SGDM) V[m].a[c] = v[m];
                if constexpr (DIAG) dd[m] = fmaf(d[m], d[m], dd[m]);
            }
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            dg.add(DIAG_D, m, dd[m]);
            if constexpr (DIAG) dg.add(DIAG_X, m, sum_sq<VEC>(X[m]));
            st_f32<VEC>(sp[0][m], e, X[m]);
            st_f32<VEC>(sp[1][m], e, U[m]);
            if constexpr (OPT != OPT_SGDM) st_f32<VEC>(sp[2][m], e, V[m]);
        }
    }
}

// One chunk of `count` elements for all MT workers: 128-bit path (with a scalar tail) when
// every pointer is aligned, scalar path otherwise.
template <int OPT, int MASK, int MT, typename GT, bool POST, bool DIAG, int NW>
__device__ __forceinline__ void process_chunk(const StepArgs &a, char *const (*sp)[MT],
                                              const float *sscale, int count, bool scalar_path,
                                              const DiagAcc<DIAG, NW> &dg) {
    const int tid = threadIdx.x;
    if (!scalar_path) {
        const int n4 = count >> 2;
        if (count == CHUNK_ELEMS) {
            // full chunk: four rounds of 256 threads x 4 elements, no bounds checks
#pragma unroll 1
            for (int r = 0; r < 4; ++r)
                process_tile<OPT, MASK, MT, GT, POST, 4, DIAG>(
                    a, sp, sscale, static_cast<long long>(r * BLOCK_THREADS + tid) * 4, dg);
        } else {
            for (int p = tid; p < n4; p += BLOCK_THREADS)
                process_tile<OPT, MASK, MT, GT, POST, 4, DIAG>(a, sp, sscale,
                                                               static_cast<long long>(p) * 4, dg);
            const int rem = count & 3;
            if (tid < rem)
                process_tile<OPT, MASK, MT, GT, POST, 1, DIAG>(a, sp, sscale, (n4 << 2) + tid, dg);
        }
    } else {
        for (int e = tid; e < count; e += BLOCK_THREADS)
            process_tile<OPT, MASK, MT, GT, POST, 1, DIAG>(a, sp, sscale, e, dg);
    }
}

// Resident blocks per SM the kernels are compiled for: three (80 registers per thread), except
// SGDM with more than four workers (all-at-once tile), which is fastest at two.  The batched
// post-average tiles moved from two to three: 0.88 -> 0.97 on ADOPT's all-sync steps (M = 8).
template <int OPT, int MT, bool POST>
__host__ __device__ constexpr int min_blocks() {
    return (MT > 4 && OPT == OPT_SGDM) ? 2 : 3;
}

template <int OPT, int MASK, int MT, typename GT, bool POST, bool DIAG>
__global__ void __launch_bounds__(BLOCK_THREADS, (min_blocks<OPT, MT, POST>()))
desloc_step_kernel(const __grid_constant__ StepArgs a) {
    __shared__ char *sp[4][MT];
    __shared__ float sscale[MT];
    __shared__ float sdiag[DIAG ? DIAG_KINDS * MT * BLOCK_THREADS : 1];
    __shared__ float swsum[DIAG ? DIAG_KINDS * MT * (BLOCK_THREADS / 32) : 1];
    const DiagAcc<DIAG, MT> dg{sdiag, swsum, 0};
    const int tid = threadIdx.x;
    if (tid < MT) sscale[tid] = a.gscale ? a.gscale[tid] : 1.f;  // published by the barriers below
    dg.clear();
    // One chunk per block as launched; a smaller grid strides over the rest.  (The loop form
    // also matters to the compiler: without it the same body needs a few spill slots.)
    for (long long c = blockIdx.x; c < a.nchunks; c += gridDim.x) {
        const Chunk ch = a.chunks[c];
        __syncthreads();  // previous chunk's readers are done with sp
        int misaligned = 0;
        if (tid < 4 * MT) {
            const int arr = tid / MT, m = tid - arr * MT;
            const long long idx = static_cast<long long>(m) * a.nt + ch.tensor;
            char *p = nullptr;
            if (arr == 0) p = reinterpret_cast<char *>(a.x[idx]) + ch.start * 4;
            if (arr == 1) p = reinterpret_cast<char *>(a.u[idx]) + ch.start * 4;
            if (arr == 2 && OPT != OPT_SGDM) p = reinterpret_cast<char *>(a.v[idx]) + ch.start * 4;
            if (arr == 3)
                p = const_cast<char *>(reinterpret_cast<const char *>(grad_ptr(a, idx))) +
                    ch.start * static_cast<long long>(sizeof(GT));
            sp[arr][m] = p;
            const unsigned need = (arr == 3 && sizeof(GT) == 2) ? 7u : 15u;
            misaligned = (reinterpret_cast<uintptr_t>(p) & need) != 0;
        }
        const int scalar_path = __syncthreads_or(misaligned);
        process_chunk<OPT, MASK, MT, GT, POST, DIAG>(a, sp, sscale, ch.count, scalar_path != 0, dg);
        if constexpr (DIAG) {
            const float total = dg.flush();
            if (tid < DIAG_KINDS * MT) {
                const int kind = tid / MT, m = tid - kind * MT;
                a.diag[(static_cast<long long>(kind) * a.M + m) * a.diag_stride + a.diag_chunk0 + c] = total;
            }
        }
    }
}

// ---- local steps with workers as separate work items (M = 1, or M > MAX_MT) -------------
// A block takes LOCAL_SLOTS consecutive chunks of one worker: their pointers are set up
// together (one dependent-load chain instead of four) and, when all of them are full and
// aligned, they are processed exactly like four replicas of one chunk on a local step.
constexpr int LOCAL_SLOTS = 4;

template <int OPT, typename GT, bool DIAG>
__global__ void __launch_bounds__(BLOCK_THREADS, 3)
desloc_local_kernel(const __grid_constant__ StepArgs a) {
    constexpr int SL = LOCAL_SLOTS;
    __shared__ char *sp[4][SL];
    __shared__ int scount[SL];
    __shared__ float sscale[SL];  // all slots belong to one worker
    __shared__ float sdiag[DIAG ? DIAG_KINDS * SL * BLOCK_THREADS : 1];
    __shared__ float swsum[DIAG ? DIAG_KINDS * SL * (BLOCK_THREADS / 32) : 1];
    const DiagAcc<DIAG, SL> dg{sdiag, swsum, 0};
    const int tid = threadIdx.x;
    const long long ngroups = (a.nchunks + SL - 1) / SL;
    const long long nitems = ngroups * a.M;
    dg.clear();
    for (long long item = blockIdx.x; item < nitems; item += gridDim.x) {
        const long long grp = item % ngroups;
        const int m0 = static_cast<int>(item / ngroups);
        __syncthreads();
        int slow = 0;
        if (tid < 4 * SL) {
            const int arr = tid / SL, sl = tid - arr * SL;
            const long long c = grp * SL + sl;
            char *p = nullptr;
            int cnt = 0;
            if (c < a.nchunks) {
                const Chunk ch = a.chunks[c];
                cnt = ch.count;
                const long long idx = static_cast<long long>(m0) * a.nt + ch.tensor;
                if (arr == 0) p = reinterpret_cast<char *>(a.x[idx]) + ch.start * 4;
                if (arr == 1) p = reinterpret_cast<char *>(a.u[idx]) + ch.start * 4;
                if (arr == 2 && OPT != OPT_SGDM) p = reinterpret_cast<char *>(a.v[idx]) + ch.start * 4;
                if (arr == 3)
                    p = const_cast<char *>(reinterpret_cast<const char *>(grad_ptr(a, idx))) +
                        ch.start * static_cast<long long>(sizeof(GT));
            }
            sp[arr][sl] = p;
            if (arr == 0) {
                scount[sl] = cnt;
                sscale[sl] = a.gscale ? a.gscale[m0] : 1.f;
            }
            const unsigned need = (arr == 3 && sizeof(GT) == 2) ? 7u : 15u;
            slow = cnt != CHUNK_ELEMS || (reinterpret_cast<uintptr_t>(p) & need) != 0;
        }
        if (!__syncthreads_or(slow)) {
#pragma unroll 1
            for (int r = 0; r < 4; ++r)
                process_tile<OPT, 0, SL, GT, false, 4, DIAG>(
                    a, sp, sscale, static_cast<long long>(r * BLOCK_THREADS + tid) * 4, dg);
        } else {
            // ragged group (a tensor's last chunk, an unaligned tensor, the list's end): slot by slot
#pragma unroll 1
            for (int sl = 0; sl < SL; ++sl) {
                const int cnt = scount[sl];
                if (cnt == 0) continue;
                char *one[4][1] = {{sp[0][sl]}, {sp[1][sl]}, {sp[2][sl]}, {sp[3][sl]}};
                unsigned long long bits = reinterpret_cast<uintptr_t>(one[0][0]) |
                                          reinterpret_cast<uintptr_t>(one[1][0]) |
                                          reinterpret_cast<uintptr_t>(one[2][0]);
                const bool mis = (bits & 15u) != 0 ||
                                 (reinterpret_cast<uintptr_t>(one[3][0]) & (sizeof(GT) == 2 ? 7u : 15u)) != 0;
                // the one-worker tile accumulates into slot `sl` of this block's diagnostics
                const DiagAcc<DIAG, SL> dg1{sdiag, swsum, sl};
                process_chunk<OPT, 0, 1, GT, false, DIAG>(a, one, sscale + sl, cnt, mis, dg1);
            }
        }
        if constexpr (DIAG) {
            const float total = dg.flush();
            if (tid < DIAG_KINDS * SL) {
                const int kind = tid / SL, sl = tid - kind * SL;
                const long long c = grp * SL + sl;
                if (c < a.nchunks)
                    a.diag[(static_cast<long long>(kind) * a.M + m0) * a.diag_stride + a.diag_chunk0 + c] = total;
            }
        }
    }
}

// Lookup of an instantiation: opt, post-average?, bf16 gradients?, MT in 1..MAX_MT, mask,
// with or without the norm diagnostics (mt = 1 with mask 0 is desloc_local_kernel).
// Returns nullptr for combinations that do not exist (sync masks with M > MAX_MT).
const void *lookup_step_kernel(int opt, bool post, bool bf16, int mt, int mask, bool diag);

// Runtime-M kernel for sync steps of M > MAX_MT; launched with (StepArgs, int mask).
const void *lookup_generic_kernel(int opt, bool post, bool bf16, int mask, bool diag);

}  // namespace desloc
