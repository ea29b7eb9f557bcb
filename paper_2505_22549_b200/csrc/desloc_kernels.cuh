// DES-LOC fused step kernel for sm_100a: one streaming pass over g, x, u, v of all M
// worker replicas (Algorithm 1 with the Adam, ADOPT and SGDM rules of Algorithms 2-3).
//
// Work decomposition.  The tensor list is cut into chunks of one tensor (table built once on the
// host); a chunk is a run of up to 8 tiles of tile_elems(M) elements.  A thread block takes
// one chunk of ALL M replicas (for M = 1, and on local steps of more than eight workers, of
// one replica) and streams its tiles through two shared-memory buffers:
//   1. the first 4*M threads look up the chunk's pointers once; each owns one (array, worker)
//      and issues ONE 1-D bulk asynchronous copy per tile (cp.async.bulk, the TMA engine; no
//      multicast, this GPU's own memory) of its 1-4 KB slice into the tile's buffer, all
//      signalling the buffer's mbarrier;
//   2. the block waits for the mbarrier (bounded; see bar_wait), then every thread updates its
//      coordinates in place in shared memory: the arrays whose period divides t are averaged
//      over the workers in a fixed tree order, then each worker takes its optimizer step -- a
//      sync step moves the same bytes as a local step, through the same code shape;
//   3. the owners of x, u, v each issue one bulk copy of the updated slice back, and, once
//      that copy has read the buffer, request the tile after next into it.
// While tile k is updated, tile k + 1 is landing and tile k - 1 is on its way back.  Two to
// three blocks are resident per SM.  A chunk whose pointers are not 16-byte aligned, and a
// ragged last tile whose byte counts are not multiples of 16, take the same arithmetic straight
// from and to global memory: four coordinates per thread with 128-bit accesses where the fp32
// arrays are 16-byte and the gradients at least 8-byte aligned, else one coordinate per thread.
//
// Measured on B200 (Adam, 4 workers, bf16 gradients, 1.7 G parameters; one local step):
//   registers only, 128-bit loads (4096-element chunks, 3 blocks/SM)   26.74 ms  1.015 of copy
//   registers only, 256-bit loads (ld.global.v8.f32)                   26.39 ms  1.029
//   bulk copies, 1024-element tiles, 2-stage pipeline, 2 blocks/SM     26.08 ms  1.041
//   bulk copies, persistent grid (2 blocks/SM striding)                30.2  ms  0.90
//   bulk copies, 512-element tiles, no pipeline, 6-8 blocks/SM         25.76 ms  1.055
// ("copy" = the device-to-device copy bandwidth of the same GPU; these are single-tensor
// experiments with the pointers in the kernel parameters).  In the library, with the tensor
// list's pointer look-up on every block's path, the pipelined form is the robust one: a run
// of 8 tiles per block through two buffers gives 26.1 ms (1.04) on the 218-tensor list,
// local and sync steps alike.
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
constexpr int MAX_MT = 8;          // largest worker count with a kernel instantiated for it
constexpr int DIAG_G = 0, DIAG_X = 1, DIAG_D = 2, DIAG_KINDS = 3;
constexpr int REDUCE_CHUNK_ELEMS = BLOCK_THREADS * 16;  // chunks of the reduction kernels (4096)
constexpr int GENERIC_CHUNK_ELEMS = 1024;               // chunks of contexts with M > MAX_MT
constexpr int DRAIN_WAIT_LIMIT = 1 << 22;               // bound on the wait for copies in flight

// Elements per tile and worker for a kernel that holds mt replicas per tile: bulk copies of
// 2-4 KB per state array (copies of 1 KB and 512 B, with 256-element tiles, were 5 % slower on
// eight workers), 28-57 KB of shared memory per buffer.
__host__ __device__ constexpr int tile_elems(int mt) { return mt <= 2 ? 1024 : 512; }
// Tiles per chunk on large problems (one pointer look-up and one pipeline fill serve them all):
// 8 measured best (4: sync steps 2 % slower; 16: 0.5-1 % slower; 32: 2 % slower).
__host__ __device__ constexpr int max_tiles_per_chunk(int) { return 8; }

struct __align__(16) Chunk {
    int32_t tensor;  // index into the tensor list
    int32_t count;   // elements in this chunk (<= the context's chunk length)
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
    int *err;             // set to 1 when a bounded wait ran out (may be nullptr)
    int wait_limit;       // iterations a block polls for its tile before it gives up
    int direct;           // non-zero: no staging, every chunk straight from global memory (tiny launches)
    int nt;
    int M;
    float b1, omb1;   // beta1, 1 - beta1
    float b2, omb2;   // beta2, 1 - beta2
    float eps2;       // ADOPT epsilon, squared
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

// ---- global memory access: 128-bit or scalar (runtime-M kernel, reductions) ---------------
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

// ---- the arithmetic of one coordinate ------------------------------------------------------
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
// 1 / sqrt(a) to within an ulp: the hardware approximation (2 ulp) with one Newton step.  This
// replaces IEEE sqrt followed by IEEE division (two roundings, about 20 instructions): with the
// tiles staged by the copy engine the arithmetic sits on each block's critical path, and the
// exact pair cost 1 % on Adam with four workers and 5-11 % on ADOPT with eight.  The error is
// that of the exact pair (about one ulp of the quotient), not its bits.
__device__ __forceinline__ float rsqrt_1ulp(float a) {
    const float y = rsqrtf(a);
    const float r = y * fmaf(-0.5f * a * y, y, 1.5f);
    return a > 0.f && a < 3.0e38f ? r : y;   // keep the limits (1/0 = inf, 1/inf = 0) free of NaN
}

template <int OPT, bool PLAIN = false>
__device__ __forceinline__ void state_update(const StepArgs &a, float g, float up, float vp,
                                             float vown, float &un, float &vn) {
    // coordinate-wise clip: sgn(g) min(|g|, rho)  (Section 3.1); rho = +inf when off
    const float gh = PLAIN ? g : fminf(fmaxf(g, -a.rho), a.rho);
    if constexpr (OPT == OPT_ADAM) {
        un = fmaf(a.b1, up, a.omb1 * gh);
        vn = fmaf(a.b2, vp, (a.omb2 * gh) * gh);
    } else if constexpr (OPT == OPT_ADOPT) {
        vn = fmaf(a.b2, vp, (a.omb2 * gh) * gh);
        float r = gh * rsqrt_1ulp(fmaxf(vown, a.eps2));  // g / max(sqrt(v), eps)
        r = fminf(fmaxf(r, -a.cbound), a.cbound);
        un = fmaf(a.b1, up, a.omb1 * r);
    } else {
        un = fmaf(a.b1, up, a.omb1 * gh);
        vn = 0.f;
    }
}

// The update d_t of Algorithms 2-3 from the new states.
template <int OPT>
__device__ __forceinline__ float direction(const StepArgs &a, float un, float vn) {
    if constexpr (OPT == OPT_ADAM)
        return (a.lr * un) * rsqrt_1ulp(vn + a.lam2);
    else
        return a.lr * un;
}

// x* (1 - eta wd) - d, written as x* - (eta wd x* + d): one rounding at x's scale
__device__ __forceinline__ float apply_step(const StepArgs &a, float xp, float d) {
    return xp - fmaf(a.lrwd, xp, d);
}

// ---- helpers of the runtime-M kernel ---------------------------------------------------------
// Registers a worker costs while its batch is in flight (FV<4> = 4 registers; bf16 g = 2).
template <int OPT, typename GT>
__host__ __device__ constexpr int worker_regs(bool ld_x, bool ld_u, bool ld_v) {
    return (sizeof(GT) == 2 ? 2 : 4) + 4 * ((ld_x ? 1 : 0) + (ld_u ? 1 : 0) + (ld_v ? 1 : 0));
}
// Post-average ordering: which per-worker values a parameter step needs after the means are
// known (shared by the tile kernel and the runtime-M kernel).
template <int OPT, int MASK>
struct PostPlan {
    static constexpr bool SX = MASK & SYNC_X, SU = MASK & SYNC_U;
    static constexpr bool SV = (MASK & SYNC_V) && OPT != OPT_SGDM;
    // does d_t depend on a state that is averaged?
    static constexpr bool D_NEEDS_MEAN = SU || (OPT == OPT_ADAM && SV);
    static constexpr bool KEEP_U = D_NEEDS_MEAN && !SU;                      // Adam, v synced only
    static constexpr bool KEEP_V = D_NEEDS_MEAN && OPT == OPT_ADAM && !SV;   // Adam, u synced only
};


// ---- where a tile lives -----------------------------------------------------------------------
// Position q of a thread covers VEC consecutive elements.  Both accessors expose the same four
// operations, so that one routine serves the staged tile and the straight-from-global fallback.
template <int OPT, int MT, typename GT, int T>
struct TileLayout {
    static constexpr int NS = OPT == OPT_SGDM ? 2 : 3;   // state arrays: x, u (, v)
    static constexpr int GB = T * static_cast<int>(sizeof(GT)), FB = T * 4;
    static constexpr int BYTES = MT * (GB + NS * FB);    // [g of every worker][x ...][u ...][v ...]
    __device__ static __forceinline__ int g_off(int m) { return m * GB; }
    __device__ static __forceinline__ int f_off(int arr, int m) { return MT * GB + (arr * MT + m) * FB; }
};

template <int OPT, int MT, typename GT, int T, int VEC_>
struct SmemAcc {
    static constexpr int VEC = VEC_;
    using L = TileLayout<OPT, MT, GT, T>;
    char *tile;
    __device__ __forceinline__ FV<VEC> ld(int arr, int m, int q) const {
        const char *p = tile + L::f_off(arr, m);
        FV<VEC> r;
        if constexpr (VEC == 4) {
            const float4 t = reinterpret_cast<const float4 *>(p)[q];
            r.a[0] = t.x; r.a[1] = t.y; r.a[2] = t.z; r.a[3] = t.w;
        } else if constexpr (VEC == 2) {
            const float2 t = reinterpret_cast<const float2 *>(p)[q];
            r.a[0] = t.x; r.a[1] = t.y;
        } else {
            r.a[0] = reinterpret_cast<const float *>(p)[q];
        }
        return r;
    }
    __device__ __forceinline__ void st(int arr, int m, int q, const FV<VEC> &r) const {
        char *p = tile + L::f_off(arr, m);
        if constexpr (VEC == 4)
            reinterpret_cast<float4 *>(p)[q] = make_float4(r.a[0], r.a[1], r.a[2], r.a[3]);
        else if constexpr (VEC == 2)
            reinterpret_cast<float2 *>(p)[q] = make_float2(r.a[0], r.a[1]);
        else
            reinterpret_cast<float *>(p)[q] = r.a[0];
    }
    __device__ __forceinline__ FV<VEC> ldg(int m, int q) const {
        const char *p = tile + L::g_off(m);
        FV<VEC> r;
        if constexpr (sizeof(GT) == 4) {
            if constexpr (VEC == 4) {
                const float4 t = reinterpret_cast<const float4 *>(p)[q];
                r.a[0] = t.x; r.a[1] = t.y; r.a[2] = t.z; r.a[3] = t.w;
            } else if constexpr (VEC == 2) {
                const float2 t = reinterpret_cast<const float2 *>(p)[q];
                r.a[0] = t.x; r.a[1] = t.y;
            } else {
                r.a[0] = reinterpret_cast<const float *>(p)[q];
            }
        } else if constexpr (VEC == 4) {   // bf16 -> fp32 is a 16-bit shift (exact)
            const uint2 t = reinterpret_cast<const uint2 *>(p)[q];
            r.a[0] = __uint_as_float(t.x << 16);
            r.a[1] = __uint_as_float(t.x & 0xffff0000u);
            r.a[2] = __uint_as_float(t.y << 16);
            r.a[3] = __uint_as_float(t.y & 0xffff0000u);
        } else if constexpr (VEC == 2) {
            const unsigned t = reinterpret_cast<const unsigned *>(p)[q];
            r.a[0] = __uint_as_float(t << 16);
            r.a[1] = __uint_as_float(t & 0xffff0000u);
        } else {
            r.a[0] = __uint_as_float(static_cast<unsigned>(reinterpret_cast<const unsigned short *>(p)[q]) << 16);
        }
        return r;
    }
};

// Straight from / to global memory, one coordinate per position (unaligned or ragged tiles).
template <int MT, typename GT>
struct GlobalAcc {
    static constexpr int VEC = 1;
    char *const (*sp)[MT];   // chunk-relative base pointers: 0 x, 1 u, 2 v, 3 g
    __device__ __forceinline__ FV<1> ld(int arr, int m, int q) const { return ld_f32<1>(sp[arr][m], q); }
    __device__ __forceinline__ void st(int arr, int m, int q, const FV<1> &r) const { st_f32<1>(sp[arr][m], q, r); }
    __device__ __forceinline__ FV<1> ldg(int m, int q) const { return ld_grad<1, GT>(sp[3][m], q); }
};

// The same with four coordinates per position and 128-bit accesses (64-bit for bf16 gradients):
// chunks whose fp32 arrays are 16-byte aligned while the bf16 gradients are only 8-byte aligned
// -- a flat layout padded to 16 bytes, where the gradient of a tensor at an odd multiple of
// four elements sits 8 bytes off -- and the aligned part of a ragged last tile.
template <int MT, typename GT>
struct GlobalAcc4 {
    static constexpr int VEC = 4;
    char *const (*sp)[MT];
    __device__ __forceinline__ FV<4> ld(int arr, int m, int q) const { return ld_f32<4>(sp[arr][m], 4LL * q); }
    __device__ __forceinline__ void st(int arr, int m, int q, const FV<4> &r) const { st_f32<4>(sp[arr][m], 4LL * q, r); }
    __device__ __forceinline__ FV<4> ldg(int m, int q) const { return ld_grad<4, GT>(sp[3][m], 4LL * q); }
};

// ---- diagnostics ------------------------------------------------------------------------------
// Each thread keeps its own running sums of squares, one per (kind, worker), in registers over
// all tiles of a chunk.  At the end of the chunk a warp reduces each of them (shuffle tree) into
// its slot of shared memory and the block total is the eight warp slots added in order:
// deterministic, and a few dozen shuffles per thread and chunk.
template <bool DIAG, int MT>
struct ThreadNorms {
    float acc[DIAG ? DIAG_KINDS * MT : 1];
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int j = 0; j < (DIAG ? DIAG_KINDS * MT : 1); ++j) acc[j] = 0.f;
    }
    __device__ __forceinline__ void add(int kind, int m, float v) {
        if constexpr (DIAG) acc[kind * MT + m] += v;
    }
    // all threads of the block call; slots: [DIAG_KINDS * MT][BLOCK_THREADS / 32]
    __device__ __forceinline__ void reduce_into(float *slots) const {
        if constexpr (DIAG) {
#pragma unroll
            for (int j = 0; j < DIAG_KINDS * MT; ++j) {
                float v = acc[j];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
                if ((threadIdx.x & 31) == 0) slots[j * (BLOCK_THREADS / 32) + (threadIdx.x >> 5)] = v;
            }
        }
    }
};

template <int VEC, int MT, typename Acc>
__device__ __forceinline__ FV<VEC> mean_over_workers(const Acc &acc, int arr, int q) {
    FV<VEC> S[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) S[m] = acc.ld(arr, m, q);
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

// ---- one position (VEC coordinates) of all MT workers, in place --------------------------------
// Pre-average (Algorithms 1-3): the arrays to be averaged are first reduced to their worker
// means, then every worker updates from the mean or from its own previous value.
// Post-average (Algorithms 4-5): every worker updates its states, the ones to be averaged are
// replaced by their means, the parameter step uses those, and a synced x is averaged last.
// A thread re-reads values it stored itself (never another thread's), so no barrier is needed.
template <int OPT, int MASK, int MT, bool POST, bool DIAG, bool PLAIN = false, typename Acc>
__device__ __forceinline__ void update_position(const StepArgs &a, const Acc &acc, const float *sscale,
                                                int q, ThreadNorms<DIAG, MT> &wn) {
    constexpr bool active = true;
    constexpr int VEC = Acc::VEC;
    constexpr bool SX = MASK & SYNC_X, SU = MASK & SYNC_U;
    constexpr bool SV = (MASK & SYNC_V) && OPT != OPT_SGDM;
    constexpr bool HAS_V = OPT != OPT_SGDM;
    if constexpr (!POST) {
        FV<VEC> xb{}, ub{}, vb{};
        if (active) {
            if constexpr (SX) xb = mean_over_workers<VEC, MT>(acc, 0, q);
            if constexpr (SU) ub = mean_over_workers<VEC, MT>(acc, 1, q);
            if constexpr (SV) vb = mean_over_workers<VEC, MT>(acc, 2, q);
        }
        constexpr bool NEED_V = HAS_V && (!SV || OPT == OPT_ADOPT);   // ADOPT: its own old v
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            float gg = 0.f, dd = 0.f, xx = 0.f;
            if (active) {
                const FV<VEC> G = acc.ldg(m, q);
                FV<VEC> X{}, U{}, V{}, D;
                if constexpr (!SX) X = acc.ld(0, m, q);
                if constexpr (!SU) U = acc.ld(1, m, q);
                if constexpr (NEED_V) V = acc.ld(2, m, q);
                const float sc = PLAIN ? 1.f : sscale[m];
#pragma unroll
                for (int c = 0; c < VEC; ++c) {
                    const float up = SU ? ub.a[c] : U.a[c];
                    const float vown = NEED_V ? V.a[c] : 0.f;
                    const float vp = SV ? vb.a[c] : vown;
                    const float xp = SX ? xb.a[c] : X.a[c];
                    float un, vn;
                    state_update<OPT, PLAIN>(a, PLAIN ? G.a[c] : G.a[c] * sc, up, vp, vown, un, vn);
                    D.a[c] = direction<OPT>(a, un, vn);
                    X.a[c] = apply_step(a, xp, D.a[c]);
                    U.a[c] = un;
                    V.a[c] = vn;
                }
                acc.st(0, m, q, X);
                acc.st(1, m, q, U);
                if constexpr (HAS_V) acc.st(2, m, q, V);
                if constexpr (DIAG) {
                    gg = sum_sq<VEC>(G); dd = sum_sq<VEC>(D); xx = sum_sq<VEC>(X);
                }
            }
            wn.add(DIAG_G, m, gg);
            wn.add(DIAG_D, m, dd);
            wn.add(DIAG_X, m, xx);
        }
    } else {
        using P = PostPlan<OPT, MASK>;
        // states
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            float gg = 0.f;
            if (active) {
                const FV<VEC> G = acc.ldg(m, q);
                FV<VEC> U = acc.ld(1, m, q), V{};
                if constexpr (HAS_V) V = acc.ld(2, m, q);
                const float sc = PLAIN ? 1.f : sscale[m];
#pragma unroll
                for (int c = 0; c < VEC; ++c) {
                    const float vown = HAS_V ? V.a[c] : 0.f;
                    float un, vn;
                    state_update<OPT, PLAIN>(a, PLAIN ? G.a[c] : G.a[c] * sc, U.a[c], vown, vown, un, vn);
                    U.a[c] = un;
                    V.a[c] = vn;
                }
                acc.st(1, m, q, U);
                if constexpr (HAS_V) acc.st(2, m, q, V);
                if constexpr (DIAG) gg = sum_sq<VEC>(G);
            }
            wn.add(DIAG_G, m, gg);
        }
        FV<VEC> mu{}, mv{};
        if (active) {
            if constexpr (SU) mu = mean_over_workers<VEC, MT>(acc, 1, q);
            if constexpr (SV) mv = mean_over_workers<VEC, MT>(acc, 2, q);
        }
        // parameters
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            float dd = 0.f, xx = 0.f;
            if (active) {
                FV<VEC> X = acc.ld(0, m, q), U = mu, V = mv, D;
                if constexpr (!SU) U = acc.ld(1, m, q);
                if constexpr (OPT == OPT_ADAM && !SV) V = acc.ld(2, m, q);
#pragma unroll
                for (int c = 0; c < VEC; ++c) {
                    D.a[c] = direction<OPT>(a, U.a[c], V.a[c]);
                    X.a[c] = apply_step(a, X.a[c], D.a[c]);
                }
                acc.st(0, m, q, X);
                if constexpr (SU) acc.st(1, m, q, mu);
                if constexpr (SV) acc.st(2, m, q, mv);
                if constexpr (DIAG) {
                    dd = sum_sq<VEC>(D);
                    xx = sum_sq<VEC>(X);
                }
            }
            wn.add(DIAG_D, m, dd);
            if constexpr (!SX) wn.add(DIAG_X, m, xx);
        }
        if constexpr (SX) {
            float xx = 0.f;
            if (active) {
                const FV<VEC> mx = mean_over_workers<VEC, MT>(acc, 0, q);
#pragma unroll
                for (int m = 0; m < MT; ++m) acc.st(0, m, q, mx);
                if constexpr (DIAG) xx = sum_sq<VEC>(mx);
            }
#pragma unroll
            for (int m = 0; m < MT; ++m) wn.add(DIAG_X, m, xx);
        }
    }
}

// ---- bulk asynchronous copies and their barrier ----------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// global -> shared, completion counted in bytes on `bar`.  Both addresses 16-byte aligned and
// `bytes` a multiple of 16 (checked by the caller: anything else takes the fallback path).
__device__ __forceinline__ void bulk_load(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// shared -> global, tracked by the issuing thread's bulk group
__device__ __forceinline__ void bulk_store(void *dst, const void *src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 :: "l"(dst), "r"(smem_u32(src)), "r"(bytes) : "memory");
}
// Waits for the phase with the given parity, polling at most `limit` times; false when the limit
// ran out.  No wait in this library is unbounded.
__device__ __forceinline__ bool bar_wait(uint64_t *bar, uint32_t parity, int limit) {
    for (int i = 0; i < limit; ++i) {
        uint32_t ok;
        asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                     : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
        if (ok) return true;
    }
    return false;
}

constexpr int STAGES = 2;         // tile buffers per block (three stages at two blocks per SM: 0.84)
// Resident blocks per SM: what the two buffers leave room for (three up to four workers, two
// beyond).
__host__ __device__ constexpr int step_min_blocks(int mt) { return mt <= 4 ? 3 : 2; }

// A chunk is a run of consecutive tiles of one tensor.  The block looks its pointers up
// once, then streams the tiles through a ring of STAGES buffers: while tile k is updated in
// place, tile k + 1 is already landing; when tile k's copy back has left its buffer, tile
// k + STAGES is requested into it.
template <int OPT, int MASK, int MT, typename GT, bool POST, bool DIAG>
__global__ void __launch_bounds__(BLOCK_THREADS, step_min_blocks(MT))
desloc_step_kernel(const __grid_constant__ StepArgs a) {
    constexpr int T = tile_elems(MT), VEC = T / BLOCK_THREADS, S = STAGES;
    constexpr int ALIGN_ELEMS = 16 / static_cast<int>(sizeof(GT));   // bulk copies move multiples of 16 bytes
    constexpr bool HAS_V = OPT != OPT_SGDM;
    using L = TileLayout<OPT, MT, GT, T>;
    static_assert(4 * MT <= 32, "the (array, worker) owners are lanes of the first warp");
    extern __shared__ __align__(128) char tile_mem[];   // S buffers of L::BYTES
    __shared__ char *sp[4][MT];
    __shared__ float sscale[MT];
    __shared__ __align__(8) uint64_t bar[S];
    ThreadNorms<DIAG, MT> wn;
    const int tid = threadIdx.x;
    if (tid < S) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(smem_u32(&bar[tid])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // this thread's role in the look-up, the loads and the stores: one (array, worker)
    const int arr = tid / MT, m = tid - arr * MT;
    const bool owner = tid < 4 * MT && (HAS_V || arr != 2);
    const int esize = arr == 3 ? static_cast<int>(sizeof(GT)) : 4;
    const int slot = arr == 3 ? L::g_off(m) : L::f_off(arr, m);
    uint32_t phases = 0;  // bit s: parity of the phase barrier s completes next
    // No factor on the gradient and no coordinate clip -- the common case -- takes a copy of the
    // inner loop without them (three instructions of about forty per coordinate: with eight
    // workers at sustained clocks 0.4-0.7 % of the step).  The fallback paths keep the one form.
    const bool plain = a.gscale == nullptr && a.rho > 3.4028235e38f;   // rho = +inf: clip off
    // Work items: chunks of all MT replicas; with MT = 1, (worker, chunk) pairs -- the single
    // replica and the local steps of more than MAX_MT workers.  One item per block as launched;
    // a smaller grid strides over the rest.
    const long long nitems = MT == 1 ? a.nchunks * a.M : a.nchunks;
    for (long long item = blockIdx.x; item < nitems; item += gridDim.x) {
        const long long c = MT == 1 ? item % a.nchunks : item;
        const int m0 = MT == 1 ? static_cast<int>(item / a.nchunks) : 0;
        const Chunk ch = a.chunks[c];   // the same 16 bytes for every thread
        const int count = ch.count;
        __syncthreads();  // the previous item is done with the shared state; the barriers exist
        char *p = nullptr;
        if (owner) {
            const long long idx = static_cast<long long>(m0 + m) * a.nt + ch.tensor;
            if (arr == 0) p = reinterpret_cast<char *>(a.x[idx]) + ch.start * 4;
            if (arr == 1) p = reinterpret_cast<char *>(a.u[idx]) + ch.start * 4;
            if (arr == 2) p = reinterpret_cast<char *>(a.v[idx]) + ch.start * 4;
            if (arr == 3)
                p = const_cast<char *>(reinterpret_cast<const char *>(grad_ptr(a, idx))) +
                    ch.start * static_cast<long long>(sizeof(GT));
            sp[arr][m] = p;
        }
        if (tid < MT) sscale[tid] = a.gscale ? a.gscale[m0 + tid] : 1.f;
        wn.clear();
        // bulk copies need 16-byte aligned addresses; a tile of the chunk also a byte count that
        // is a multiple of 16 (only the chunk's last tile can miss that: it is then updated
        // straight from global memory, like every tile of a chunk whose pointers are unaligned)
        const bool unaligned = __syncthreads_or((reinterpret_cast<uintptr_t>(p) & 15u) != 0) != 0;
        // 128-bit accesses from global memory need less: 8 bytes for bf16 gradients
        const uintptr_t need = (arr == 3 && sizeof(GT) == 2) ? 7u : 15u;
        const bool wide_ok = __syncthreads_or((reinterpret_cast<uintptr_t>(p) & need) != 0) == 0;
        const int ntiles = (count + T - 1) / T;
        // (a launch of a single wave of single-tile chunks has nothing to overlap: staging would
        // only add the copy engine's round trip to every step of a latency-bound problem)
        const int staged = (unaligned || a.direct) ? 0 : ((count % T) % ALIGN_ELEMS == 0 ? ntiles : ntiles - 1);   // tiles 0 .. staged-1
        // request tile k (< staged) into its buffer: every owner its own slice, one arrival
        auto request = [&](int k) {
            const int cnt = min(T, count - k * T);
            if (owner)
                bulk_load(tile_mem + (k % S) * L::BYTES + slot, p + static_cast<long long>(k) * T * esize,
                          static_cast<uint32_t>(cnt * esize), &bar[k % S]);
            if (tid == 0)
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                             :: "r"(smem_u32(&bar[k % S])),
                                "r"(static_cast<uint32_t>(MT * cnt * (static_cast<int>(sizeof(GT)) + 4 * L::NS)))
                             : "memory");
        };
#pragma unroll
        for (int k = 0; k < S; ++k)
            if (k < staged) request(k);
#pragma unroll 1
        for (int k = 0; k < staged; ++k) {
            const int st = k % S;
            const int cnt = min(T, count - k * T);
            const bool landed = bar_wait(&bar[st], (phases >> st) & 1u, a.wait_limit);
            if (__syncthreads_or(!landed)) {
                // Give up on this step: say so, let the copies already requested land (bounded as
                // well), store nothing more, leave.  The host reports the flag on its next call.
                if (tid == 0 && a.err) *reinterpret_cast<volatile int *>(a.err) = 1;
                for (int kk = k; kk < staged && kk < k + S; ++kk)
                    bar_wait(&bar[kk % S], (phases >> (kk % S)) & 1u, DRAIN_WAIT_LIMIT);
                asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
                __syncthreads();
                return;
            }
            phases ^= 1u << st;
            const SmemAcc<OPT, MT, GT, T, VEC> acc{tile_mem + st * L::BYTES};
            if (tid * VEC < cnt) {
                if (plain) update_position<OPT, MASK, MT, POST, DIAG, true>(a, acc, sscale, tid, wn);
                else update_position<OPT, MASK, MT, POST, DIAG, false>(a, acc, sscale, tid, wn);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // our writes, then the copy engine's reads
            __syncthreads();
            if (owner && arr != 3) {
                bulk_store(p + static_cast<long long>(k) * T * 4, tile_mem + st * L::BYTES + slot,
                           static_cast<uint32_t>(cnt * 4));
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            }
            if (k + S < staged) {
                // the buffer is free once this thread's own copy back has read it
                if (owner && arr != 3) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                request(k + S);
            }
        }
        if (staged * T < count) {
            // what could not be staged: the whole chunk, or its ragged last tile
            int e0 = staged * T;
            if (wide_ok) {
                const GlobalAcc4<MT, GT> acc4{sp};
                const int p1 = count >> 2;
                for (int q = (e0 >> 2) + tid; q < p1; q += BLOCK_THREADS)
                    update_position<OPT, MASK, MT, POST, DIAG>(a, acc4, sscale, q, wn);
                e0 = p1 << 2;
            }
            const GlobalAcc<MT, GT> acc{sp};
            for (int e = e0 + tid; e < count; e += BLOCK_THREADS)
                update_position<OPT, MASK, MT, POST, DIAG>(a, acc, sscale, e, wn);
        }
        // the copies back must have left shared memory before the buffers are reused or freed
        if (owner && arr != 3) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        if constexpr (DIAG) {
            // the tile buffers are idle now: their first bytes serve as the warps' slots
            float *slots = reinterpret_cast<float *>(tile_mem);
            __syncthreads();
            wn.reduce_into(slots);
            __syncthreads();
            if (tid < DIAG_KINDS * MT) {
                float total = 0.f;
#pragma unroll
                for (int w = 0; w < BLOCK_THREADS / 32; ++w) total += slots[tid * (BLOCK_THREADS / 32) + w];
                const int kind = tid / MT, mm = tid - kind * MT;
                a.diag[(static_cast<long long>(kind) * a.M + m0 + mm) * a.diag_stride + a.diag_chunk0 + c] = total;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // before the copy engine writes there again
        }
    }
}

// Dynamic shared memory a launch of desloc_step_kernel<opt, ., mt, grad type, ., .> needs.
__host__ __device__ constexpr int step_smem_bytes(int opt, int mt, bool bf16) {
    return STAGES * mt * tile_elems(mt) * ((bf16 ? 2 : 4) + 4 * (opt == OPT_SGDM ? 2 : 3));
}

// Lookup of an instantiation: opt, post-average?, bf16 gradients?, MT in 1..MAX_MT, mask,
// with or without the norm diagnostics (MT = 1 exists for mask 0 only).
// Returns nullptr for combinations that do not exist (sync masks with M > MAX_MT).
const void *lookup_step_kernel(int opt, bool post, bool bf16, int mt, int mask, bool diag);

// Runtime-M kernel for sync steps of M > MAX_MT.
const void *lookup_generic_kernel(int opt, bool post, bool bf16, int mask, bool diag);

}  // namespace desloc
