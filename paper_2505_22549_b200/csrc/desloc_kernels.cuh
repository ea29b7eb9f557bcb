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
// Every thread issues all loads of its tile (MT workers x UN positions x 4 arrays, 128-bit
// where aligned) before the first use, so that enough bytes are in flight to cover HBM
// latency; the arithmetic is fp32.  Tensors whose pointers are not 16-byte aligned and the
// last (numel mod 4) elements of a tensor take the scalar instantiation of the same code.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

// Tuning of the MT > 4 instantiations (measured on B200, 360 M parameters x 8 workers): Adam
// and ADOPT run the batched tile below at three blocks per SM (97 % of copy bandwidth against
// 94-95 % for the all-at-once tile, which spills at 128 registers); SGDM, with one state less,
// is fastest all-at-once at two blocks per SM (98 %).
#ifndef DESLOC_SPLIT_LARGE_M
#define DESLOC_SPLIT_LARGE_M 1
#endif
// Worker batches of the MT > 4 tile: balanced (3+2, 3+3, 4+3, 4+4) instead of 4 + rest; lifts the
// all-sync steps of M = 5, 6 from 0.89-0.92 to 0.98 of the copy bandwidth.
#ifndef DESLOC_BALANCED_BATCHES
#define DESLOC_BALANCED_BATCHES 1
#endif
#ifndef DESLOC_SPLIT_LARGE_M_POST
#define DESLOC_SPLIT_LARGE_M_POST 1
#endif
// Cache policy of the state and gradient accesses (0 = .cs evict-first, 1 = default,
// 2 = .cg / L2 only).  Measured on B200: plain loads with plain stores are 2 % faster than
// evict-first on every workload (27.0 against 27.55 ms on 1.7 B x 4); changing only one side
// gains nothing.
#ifndef DESLOC_LD_MODE
#define DESLOC_LD_MODE 1
#endif
#ifndef DESLOC_ST_MODE
#define DESLOC_ST_MODE 1
#endif
// 1: hardware reciprocal square root (about 2 ulp) instead of IEEE sqrt + division in the Adam
// direction and the ADOPT normaliser.
#ifndef DESLOC_FAST_MATH
#define DESLOC_FAST_MATH 0
#endif
#ifndef DESLOC_BLOCK_THREADS
#define DESLOC_BLOCK_THREADS 256
#endif
#ifndef DESLOC_MINB_SMALL_M
#define DESLOC_MINB_SMALL_M 3
#endif
#ifndef DESLOC_MINB_POST_LARGE_M
#define DESLOC_MINB_POST_LARGE_M 2
#endif
#ifndef DESLOC_MINB_LARGE_M
#define DESLOC_MINB_LARGE_M 3
#endif

namespace desloc {

constexpr int OPT_ADAM = 0, OPT_ADOPT = 1, OPT_SGDM = 2;
constexpr int SYNC_X = 1, SYNC_U = 2, SYNC_V = 4;
constexpr int BLOCK_THREADS = DESLOC_BLOCK_THREADS;
constexpr int CHUNK_ELEMS = BLOCK_THREADS * 16;  // 256 threads x 4 elements x 4 rounds = 4096
constexpr int MAX_MT = 8;          // largest worker count with a register-resident kernel

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

// ---- global memory access: 128-bit or scalar, cache policy per DESLOC_LD/ST_MODE ----------
template <typename T>
__device__ __forceinline__ T ld_stream(const T *p) {
#if DESLOC_LD_MODE == 0
    return __ldcs(p);
#elif DESLOC_LD_MODE == 1
    return *p;
#else
    return __ldcg(p);
#endif
}

template <typename T>
__device__ __forceinline__ void st_stream(T *p, const T &v) {
#if DESLOC_ST_MODE == 0
    __stcs(p, v);
#elif DESLOC_ST_MODE == 1
    *p = v;
#else
    __stcg(p, v);
#endif
}

template <int VEC>
__device__ __forceinline__ FV<VEC> ld_f32(const char *base, long long elem) {
    FV<VEC> r;
    if constexpr (VEC == 4) {
        const float4 t = ld_stream(reinterpret_cast<const float4 *>(base) + (elem >> 2));
        r.a[0] = t.x; r.a[1] = t.y; r.a[2] = t.z; r.a[3] = t.w;
    } else {
        r.a[0] = ld_stream(reinterpret_cast<const float *>(base) + elem);
    }
    return r;
}

template <int VEC>
__device__ __forceinline__ void st_f32(char *base, long long elem, const FV<VEC> &r) {
    if constexpr (VEC == 4) {
        st_stream(reinterpret_cast<float4 *>(base) + (elem >> 2),
                  make_float4(r.a[0], r.a[1], r.a[2], r.a[3]));
    } else {
        st_stream(reinterpret_cast<float *>(base) + elem, r.a[0]);
    }
}

template <int VEC, typename GT>
__device__ __forceinline__ FV<VEC> ld_grad(const char *base, long long elem) {
    FV<VEC> r;
    if constexpr (sizeof(GT) == 4) {
        r = ld_f32<VEC>(base, elem);
    } else if constexpr (VEC == 4) {
        // four bf16 in 8 bytes; bf16 -> fp32 is a 16-bit shift (exact)
        const uint2 t = ld_stream(reinterpret_cast<const uint2 *>(base) + (elem >> 2));
        r.a[0] = __uint_as_float(t.x << 16);
        r.a[1] = __uint_as_float(t.x & 0xffff0000u);
        r.a[2] = __uint_as_float(t.y << 16);
        r.a[3] = __uint_as_float(t.y & 0xffff0000u);
    } else {
        const unsigned short t = ld_stream(reinterpret_cast<const unsigned short *>(base) + elem);
        r.a[0] = __uint_as_float(static_cast<unsigned>(t) << 16);
    }
    return r;
}

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
template <int OPT>
__device__ __forceinline__ void state_update(const StepArgs &a, float g, float up, float vp,
                                             float vown, float &un, float &vn) {
    // coordinate-wise clip: sgn(g) min(|g|, rho)  (Section 3.1); rho = +inf when off
    const float gh = fminf(fmaxf(g, -a.rho), a.rho);
    if constexpr (OPT == OPT_ADAM) {
        un = fmaf(a.b1, up, a.omb1 * gh);
        vn = fmaf(a.b2, vp, (a.omb2 * gh) * gh);
    } else if constexpr (OPT == OPT_ADOPT) {
        vn = fmaf(a.b2, vp, (a.omb2 * gh) * gh);
#if DESLOC_FAST_MATH
        float r = gh * rsqrtf(fmaxf(vown, a.eps * a.eps));
#else
        float r = gh / fmaxf(sqrtf(vown), a.eps);
#endif
        r = fminf(fmaxf(r, -a.cbound), a.cbound);
        un = fmaf(a.b1, up, a.omb1 * r);
    } else {
        un = fmaf(a.b1, up, a.omb1 * gh);
        vn = 0.f;
    }
}

// One worker's parameter step from base xp with the new states.
template <int OPT>
__device__ __forceinline__ float param_step(const StepArgs &a, float xp, float un, float vn) {
    float d;
    if constexpr (OPT == OPT_ADAM) {
#if DESLOC_FAST_MATH
        d = (a.lr * un) * rsqrtf(vn + a.lam2);
#else
        d = (a.lr * un) / sqrtf(vn + a.lam2);
#endif
    } else {
        d = a.lr * un;
    }
    // x* (1 - eta wd) - d, written as x* - (eta wd x* + d): one rounding at x's scale
    return xp - fmaf(a.lrwd, xp, d);
}

template <int OPT, int MASK, int MT, bool POST>
__device__ __forceinline__ void update_coord(const StepArgs &a, const float (&g)[MT],
                                             float (&x)[MT], float (&u)[MT], float (&v)[MT]) {
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
        xn[m] = param_step<OPT>(a, xp, un[m], vn[m]);
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

// ---- pre-average tile for many workers: means first, then workers in batches -------------
// With more than four replicas per thread the all-at-once tile needs more registers than two
// resident blocks allow.  Here the arrays to be averaged are loaded for all MT workers and
// reduced to their means; the per-worker phase then runs over batches of up to four workers,
// loading only what is not averaged (ADOPT also its own v).  Same loads, same arithmetic, same
// summation tree -- bitwise the same result as process_tile.
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

template <int OPT, int MASK, int MT, typename GT, int VEC, int M0, int B>
__device__ __forceinline__ void worker_batch(const StepArgs &a, char *const (*sp)[MT],
                                             const float *sscale, long long e,
                                             const FV<VEC> &xb, const FV<VEC> &ub,
                                             const FV<VEC> &vb) {
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
#pragma unroll
        for (int c = 0; c < VEC; ++c) {
            const float up = SU ? ub.a[c] : U[b].a[c];
            const float vown = NEED_V ? V[b].a[c] : 0.f;
            const float vp = SV ? vb.a[c] : vown;
            const float xp = SX ? xb.a[c] : X[b].a[c];
            float un, vn;
            state_update<OPT>(a, G[b].a[c] * sscale[M0 + b], up, vp, vown, un, vn);
            X[b].a[c] = param_step<OPT>(a, xp, un, vn);
            U[b].a[c] = un;
            V[b].a[c] = vn;
        }
        st_f32<VEC>(sp[0][M0 + b], e, X[b]);
        st_f32<VEC>(sp[1][M0 + b], e, U[b]);
        if constexpr (OPT != OPT_SGDM) st_f32<VEC>(sp[2][M0 + b], e, V[b]);
    }
}

template <int OPT, int MASK, int MT, typename GT, int VEC>
__device__ __forceinline__ void process_tile_split(const StepArgs &a, char *const (*sp)[MT],
                                                   const float *sscale, long long e) {
    FV<VEC> xb{}, ub{}, vb{};
    if constexpr (MASK & SYNC_X) xb = mean_over_workers<VEC, MT>(sp[0], e);
    if constexpr (MASK & SYNC_U) ub = mean_over_workers<VEC, MT>(sp[1], e);
    if constexpr ((MASK & SYNC_V) && OPT != OPT_SGDM) vb = mean_over_workers<VEC, MT>(sp[2], e);
    constexpr int B0 = DESLOC_BALANCED_BATCHES ? (MT + 1) / 2 : 4;
    worker_batch<OPT, MASK, MT, GT, VEC, 0, B0>(a, sp, sscale, e, xb, ub, vb);
    worker_batch<OPT, MASK, MT, GT, VEC, B0, MT - B0>(a, sp, sscale, e, xb, ub, vb);
}

// ---- post-average tile for many workers ---------------------------------------------------
// Averages are taken over the UPDATED values, so every worker's new u, v must exist before any
// parameter step.  Phase A updates the states four workers at a time and keeps them; phase B
// forms the means of the synced ones; phase C loads x four workers at a time and steps it; a
// synced x is averaged last.  Same arithmetic and summation tree as process_tile.
template <int OPT, int MT, typename GT, int VEC, int M0, int B>
__device__ __forceinline__ void post_states_batch(const StepArgs &a, char *const (*sp)[MT],
                                                  const float *sscale, long long e,
                                                  FV<VEC> (&UN)[MT], FV<VEC> (&VN)[MT]) {
    FV<VEC> G[B], U[B], V[B];
#pragma unroll
    for (int b = 0; b < B; ++b) {
        G[b] = ld_grad<VEC, GT>(sp[3][M0 + b], e);
        U[b] = ld_f32<VEC>(sp[1][M0 + b], e);
        if constexpr (OPT != OPT_SGDM) V[b] = ld_f32<VEC>(sp[2][M0 + b], e);
    }
#pragma unroll
    for (int b = 0; b < B; ++b) {
#pragma unroll
        for (int c = 0; c < VEC; ++c) {
            const float vown = OPT != OPT_SGDM ? V[b].a[c] : 0.f;
            state_update<OPT>(a, G[b].a[c] * sscale[M0 + b], U[b].a[c], vown, vown,
                              UN[M0 + b].a[c], VN[M0 + b].a[c]);
        }
    }
}

template <int OPT, int MASK, int MT, int VEC, int M0, int B>
__device__ __forceinline__ void post_params_batch(const StepArgs &a, char *const (*sp)[MT],
                                                  long long e, const FV<VEC> (&UN)[MT],
                                                  const FV<VEC> (&VN)[MT], FV<VEC> (&XN)[MT]) {
    FV<VEC> X[B];
#pragma unroll
    for (int b = 0; b < B; ++b) X[b] = ld_f32<VEC>(sp[0][M0 + b], e);
#pragma unroll
    for (int b = 0; b < B; ++b) {
#pragma unroll
        for (int c = 0; c < VEC; ++c)
            XN[M0 + b].a[c] = param_step<OPT>(a, X[b].a[c], UN[M0 + b].a[c], VN[M0 + b].a[c]);
        if constexpr (!(MASK & SYNC_X)) st_f32<VEC>(sp[0][M0 + b], e, XN[M0 + b]);
        st_f32<VEC>(sp[1][M0 + b], e, UN[M0 + b]);
        if constexpr (OPT != OPT_SGDM) st_f32<VEC>(sp[2][M0 + b], e, VN[M0 + b]);
    }
}

template <int VEC, int MT>
__device__ __forceinline__ void replace_by_mean(FV<VEC> (&S)[MT]) {
#pragma unroll
    for (int c = 0; c < VEC; ++c) {
        float s[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) s[m] = S[m].a[c];
        const float mean = mean_of<MT>(s);
#pragma unroll
        for (int m = 0; m < MT; ++m) S[m].a[c] = mean;
    }
}

template <int OPT, int MASK, int MT, typename GT, int VEC>
__device__ __forceinline__ void process_tile_split_post(const StepArgs &a, char *const (*sp)[MT],
                                                        const float *sscale, long long e) {
    FV<VEC> UN[MT], VN[MT], XN[MT];
    post_states_batch<OPT, MT, GT, VEC, 0, 4>(a, sp, sscale, e, UN, VN);
    post_states_batch<OPT, MT, GT, VEC, 4, MT - 4>(a, sp, sscale, e, UN, VN);
    if constexpr (MASK & SYNC_U) replace_by_mean<VEC, MT>(UN);
    if constexpr ((MASK & SYNC_V) && OPT != OPT_SGDM) replace_by_mean<VEC, MT>(VN);
    post_params_batch<OPT, MASK, MT, VEC, 0, 4>(a, sp, e, UN, VN, XN);
    post_params_batch<OPT, MASK, MT, VEC, 4, MT - 4>(a, sp, e, UN, VN, XN);
    if constexpr (MASK & SYNC_X) {
        replace_by_mean<VEC, MT>(XN);
#pragma unroll
        for (int m = 0; m < MT; ++m) st_f32<VEC>(sp[0][m], e, XN[m]);
    }
}

// ---- one thread's tile: MT workers x UN positions of VEC elements ------------------------
// sp[arr][m] are chunk-relative base pointers in shared memory (arr: 0 x, 1 u, 2 v, 3 g).
// Position j covers elements e0 + j * pstride .. + VEC - 1; positions >= npos are skipped.
template <int OPT, int MASK, int MT, typename GT, bool POST, int VEC, int UN, bool FULL>
__device__ __forceinline__ void process_tile(const StepArgs &a, char *const (*sp)[MT],
                                             const float *sscale, long long e0, int pstride,
                                             int npos) {
#if DESLOC_SPLIT_LARGE_M
    if constexpr (!POST && MT > 4 && UN == 1 && OPT != OPT_SGDM) {
        if (FULL || npos > 0) process_tile_split<OPT, MASK, MT, GT, VEC>(a, sp, sscale, e0);
        return;
    }
#endif
#if DESLOC_SPLIT_LARGE_M_POST
    // measured: faster for Adam (0.97-0.99 of copy bandwidth against 0.95), slower for ADOPT
    if constexpr (POST && MT > 4 && UN == 1 && MASK != 0 && OPT == OPT_ADAM) {
        if (FULL || npos > 0) process_tile_split_post<OPT, MASK, MT, GT, VEC>(a, sp, sscale, e0);
        return;
    }
#endif
    FV<VEC> G[UN][MT], X[UN][MT], U[UN][MT], V[UN][MT];
#pragma unroll
    for (int j = 0; j < UN; ++j) {
        if (FULL || j < npos) {
            const long long e = e0 + static_cast<long long>(j) * pstride;
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                G[j][m] = ld_grad<VEC, GT>(sp[3][m], e);
                X[j][m] = ld_f32<VEC>(sp[0][m], e);
                U[j][m] = ld_f32<VEC>(sp[1][m], e);
                if constexpr (OPT != OPT_SGDM) V[j][m] = ld_f32<VEC>(sp[2][m], e);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < UN; ++j) {
        if (FULL || j < npos) {
            const long long e = e0 + static_cast<long long>(j) * pstride;
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                float g[MT], x[MT], u[MT], v[MT];
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    g[m] = G[j][m].a[c] * sscale[m];
                    x[m] = X[j][m].a[c];
                    u[m] = U[j][m].a[c];
                    v[m] = (OPT != OPT_SGDM) ? V[j][m].a[c] : 0.f;
                }
                update_coord<OPT, MASK, MT, POST>(a, g, x, u, v);
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    X[j][m].a[c] = x[m];
                    U[j][m].a[c] = u[m];
                    if constexpr (OPT != OPT_SGDM) V[j][m].a[c] = v[m];
                }
            }
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                st_f32<VEC>(sp[0][m], e, X[j][m]);
                st_f32<VEC>(sp[1][m], e, U[j][m]);
                if constexpr (OPT != OPT_SGDM) st_f32<VEC>(sp[2][m], e, V[j][m]);
            }
        }
    }
}

// Positions per thread and tile: one.  (Two positions for MT = 2 spilled under the register
// cap of three blocks per SM; one worker at a time, MT = 1, only occurs on the ragged path of
// desloc_local_kernel, which must stay light on registers next to the fast path.)
template <int MT>
struct UnrollFor {
    static constexpr int value = 1;
};

// One chunk of `count` elements for all MT workers: 128-bit path (with a scalar tail) when
// every pointer is aligned, scalar path otherwise.
template <int OPT, int MASK, int MT, typename GT, bool POST>
__device__ __forceinline__ void process_chunk(const StepArgs &a, char *const (*sp)[MT],
                                              const float *sscale, int count, bool scalar_path) {
    constexpr int UN = UnrollFor<MT>::value;
    const int tid = threadIdx.x;
    if (!scalar_path) {
        if (count == CHUNK_ELEMS) {
            // full chunk: 4 * UN * 256 * (4 / UN) elements, no bounds checks
#pragma unroll 1
            for (int r = 0; r < 4 / UN; ++r)
                process_tile<OPT, MASK, MT, GT, POST, 4, UN, true>(
                    a, sp, sscale, static_cast<long long>(r * UN * BLOCK_THREADS + tid) * 4,
                    BLOCK_THREADS * 4, UN);
        } else {
            const int n4 = count >> 2;
            for (int p0 = tid; p0 < n4; p0 += UN * BLOCK_THREADS) {
                const int left = (n4 - p0 + BLOCK_THREADS - 1) / BLOCK_THREADS;
                process_tile<OPT, MASK, MT, GT, POST, 4, UN, false>(
                    a, sp, sscale, static_cast<long long>(p0) * 4, BLOCK_THREADS * 4,
                    left < UN ? left : UN);
            }
            const int rem = count & 3;
            if (tid < rem)
                process_tile<OPT, MASK, MT, GT, POST, 1, 1, true>(a, sp, sscale, (n4 << 2) + tid, 0, 1);
        }
    } else {
        for (int e = tid; e < count; e += BLOCK_THREADS)
            process_tile<OPT, MASK, MT, GT, POST, 1, 1, true>(a, sp, sscale, e, 0, 1);
    }
}

template <int OPT, int MASK, int MT, typename GT, bool POST>
__global__ void __launch_bounds__(BLOCK_THREADS, (MT <= 4 ? DESLOC_MINB_SMALL_M : ((OPT == OPT_SGDM || POST) ? DESLOC_MINB_POST_LARGE_M : DESLOC_MINB_LARGE_M)))
desloc_step_kernel(const __grid_constant__ StepArgs a) {
    __shared__ char *sp[4][MT];
    __shared__ float sscale[MT];
    const int tid = threadIdx.x;
    if (tid < MT) sscale[tid] = a.gscale ? a.gscale[tid] : 1.f;  // published by the barriers below
    for (long long c = blockIdx.x; c < a.nchunks; c += gridDim.x) {
        constexpr int m0 = 0;
        const Chunk ch = a.chunks[c];
        __syncthreads();  // previous chunk's readers are done with sp
        int misaligned = 0;
        if (tid < 4 * MT) {
            const int arr = tid / MT, m = tid - arr * MT;
            const long long idx = static_cast<long long>(m0 + m) * a.nt + ch.tensor;
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
        process_chunk<OPT, MASK, MT, GT, POST>(a, sp, sscale, ch.count, scalar_path != 0);
    }
}

// ---- local steps with workers as separate work items (M = 1, or M > MAX_MT) -------------
// A block takes LOCAL_SLOTS consecutive chunks of one worker: their pointers are set up
// together (one dependent-load chain instead of four) and, when all of them are full and
// aligned, they are processed exactly like four replicas of one chunk on a local step.
constexpr int LOCAL_SLOTS = 4;

template <int OPT, typename GT>
__global__ void __launch_bounds__(BLOCK_THREADS, 3)
desloc_local_kernel(const __grid_constant__ StepArgs a) {
    constexpr int SL = LOCAL_SLOTS;
    __shared__ char *sp[4][SL];
    __shared__ int scount[SL];
    __shared__ float sscale[SL];  // all slots belong to one worker
    const int tid = threadIdx.x;
    const long long ngroups = (a.nchunks + SL - 1) / SL;
    const long long nitems = ngroups * a.M;
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
                process_tile<OPT, 0, SL, GT, false, 4, 1, true>(
                    a, sp, sscale, static_cast<long long>(r * BLOCK_THREADS + tid) * 4,
                    BLOCK_THREADS * 4, 1);
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
                process_chunk<OPT, 0, 1, GT, false>(a, one, sscale + sl, cnt, mis);
            }
        }
    }
}

// Lookup of an instantiation: opt, post-average?, bf16 gradients?, MT in 1..MAX_MT, mask
// (mt = 1 with mask 0 is desloc_local_kernel).
// Returns nullptr for combinations that do not exist (sync masks with M > MAX_MT).
const void *lookup_step_kernel(int opt, bool post, bool bf16, int mt, int mask);

// Runtime-M kernel for sync steps of M > MAX_MT; launched with (StepArgs, int mask).
const void *lookup_generic_kernel(int opt, bool post, bool bf16, int mask);

}  // namespace desloc
