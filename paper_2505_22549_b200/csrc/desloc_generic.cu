// DES-LOC step for worker counts beyond the register-resident kernels (M > MAX_MT) on steps
// that average something.  Same update as desloc_step_kernel, runtime M, compile-time mask.
// Worker sums run in the order m = 0..M-1 as compensated fp32 sums (see WorkerSum): exact for
// equal replicas, and within an ulp of a sequential fp64 reference.
//
// A block takes one chunk and first puts the chunk-relative pointers of all M workers into
// shared memory, so that the per-position loops read them as broadcasts instead of chasing the
// pointer tables in global memory.  Per position (4 elements per thread):
//   pre-average   the arrays to be averaged are summed one array at a time, eight workers'
//                 loads in flight; then the workers are updated in batches sized to the
//                 register budget, loading only what was not averaged (ADOPT also its own v).
//                 Each array is read once and written once.
//   post-average  phase A updates the states batch by batch, sums the ones to be averaged and
//                 stores the others; the parameter step runs in phase A when d_t uses only the
//                 worker's own states, otherwise in phase B once the means are known.  Only
//                 when Adam averages exactly one of u, v does phase B re-read the other one
//                 (just written, so it is served from cache).
#include "desloc_kernels.cuh"

namespace desloc {

namespace {

constexpr int GEN_MAX_M = 256;    // worker pointers staged per chunk (= the context's limit)
// Measured on B200 (134.5 M parameters x 16 workers, fraction of the copy bandwidth on all-sync
// steps): three blocks per SM with small batches 0.96; two blocks with batches twice as large
// 0.85; fp64 worker sums 0.87 and IEEE sqrt / division instead of the hardware reciprocal
// square root 0.87 (this kernel is bound by instruction issue: ~75 instructions per
// worker-coordinate with those, ~45 without).
constexpr int GEN_MIN_BLOCKS = 3;   // 80 registers per thread
constexpr int GEN_BUDGET = 24;      // registers a batch of workers may hold in flight

// Workers per batch of the update loops: what fits in `budget` registers -- 1, 2 or 4 (a power
// of two, so that a full batch can be summed as a tree).
__host__ __device__ constexpr int gen_batch(int per_worker, int budget) {
    const int b = budget / per_worker;
    return b < 2 ? 1 : (b < 4 ? 2 : 4);
}

// Sum over the workers of one coordinate group, in the order m = 0..M-1, as a compensated fp32
// sum ("two-sum"): the running sum and the exact rounding error of every addition are both
// kept, so the pair carries about 48 bits -- the accuracy of an fp64 sum without the fp64 pipe,
// which made an all-sync step 10 % slower here.  The mean divides the pair by M with one
// correction step, and is exact (the value itself) when all M replicas are equal.
template <int VEC>
struct WorkerSum {
    float s[VEC], err[VEC];
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int c = 0; c < VEC; ++c) s[c] = err[c] = 0.f;
    }
    __device__ __forceinline__ void add(const FV<VEC> &v) {
#pragma unroll
        for (int c = 0; c < VEC; ++c) {
            const float x = v.a[c];
            const float t = s[c] + x;
            const float bp = t - s[c];
            err[c] += (s[c] - (t - bp)) + (x - bp);  // exact error of t = s + x
            s[c] = t;
        }
    }
    __device__ __forceinline__ FV<VEC> mean(int M) const {
        const float mf = static_cast<float>(M);
        FV<VEC> r;
#pragma unroll
        for (int c = 0; c < VEC; ++c) {
            const float hi = s[c] + err[c];
            const float lo = err[c] - (hi - s[c]);          // hi + lo = s + err
            const float q = hi / mf;
            const float rem = fmaf(-q, mf, hi) + lo;        // what q * M still misses
            r.a[c] = q + rem / mf;
        }
        return r;
    }
    // A batch of B consecutive workers (B a power of two) of which the first n exist.  A full
    // batch is summed as a binary tree first (exact when its values are equal) and enters the
    // running sum as one value; a partial batch enters value by value.
    template <int B>
    __device__ __forceinline__ void add_batch(const FV<VEC> (&v)[B], int n) {
        static_assert((B & (B - 1)) == 0, "batches are powers of two");
        if (n >= B) {
            FV<VEC> t;
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                float q[B];
#pragma unroll
                for (int j = 0; j < B; ++j) q[j] = v[j].a[c];
                t.a[c] = tree_sum<0, B, B>(q);
            }
            add(t);
        } else {
#pragma unroll
            for (int j = 0; j < B; ++j)
                if (j < n) add(v[j]);
        }
    }
};

// Worker means of the arrays selected by SX, SU, SV in one pass over the workers: the loads of
// a batch of workers (all selected arrays) are issued together -- four workers for one array,
// two for two or three -- and then added in worker order, one accumulator per array.
template <int VEC, bool SX, bool SU, bool SV>
__device__ __forceinline__ void means_of_workers(char *const (*sp)[GEN_MAX_M], int M, long long e,
                                                 bool active, FV<VEC> &xb, FV<VEC> &ub, FV<VEC> &vb) {
    constexpr int NS = (SX ? 1 : 0) + (SU ? 1 : 0) + (SV ? 1 : 0);
    constexpr int NB = NS == 1 ? 4 : 2;
    WorkerSum<VEC> ax, au, av;
    ax.clear(); au.clear(); av.clear();
#pragma unroll 1
    for (int m0 = 0; m0 < M; m0 += NB) {
        FV<VEC> bx[NB], bu[NB], bv[NB];
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            if (active && m0 + j < M) {
                if constexpr (SX) bx[j] = ld_f32<VEC>(sp[0][m0 + j], e);
                if constexpr (SU) bu[j] = ld_f32<VEC>(sp[1][m0 + j], e);
                if constexpr (SV) bv[j] = ld_f32<VEC>(sp[2][m0 + j], e);
            }
        }
        if (active) {
            if constexpr (SX) ax.template add_batch<NB>(bx, M - m0);
            if constexpr (SU) au.template add_batch<NB>(bu, M - m0);
            if constexpr (SV) av.template add_batch<NB>(bv, M - m0);
        }
    }
    if constexpr (SX) xb = ax.mean(M);
    if constexpr (SU) ub = au.mean(M);
    if constexpr (SV) vb = av.mean(M);
}

// Diagnostics with a runtime worker count: a warp reduces each (kind, worker) value at once
// and lane 0 adds it to the warp's own row of shared memory, in position order.
template <bool DIAG>
struct WarpDiag {
    float *rows;  // [BLOCK_THREADS / 32][DIAG_KINDS][GEN_MAX_M]
    __device__ __forceinline__ void add(int kind, int m, float v) const {
        if constexpr (DIAG) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
            if ((threadIdx.x & 31) == 0)
                rows[((threadIdx.x >> 5) * DIAG_KINDS + kind) * GEN_MAX_M + m] += v;
        }
    }
    // the same value for every worker (a synced x): one reduction, M additions by lane 0
    __device__ __forceinline__ void add_all(int kind, int M, float v) const {
        if constexpr (DIAG) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
            if ((threadIdx.x & 31) == 0) {
                float *row = rows + ((threadIdx.x >> 5) * DIAG_KINDS + kind) * GEN_MAX_M;
                for (int m = 0; m < M; ++m) row[m] += v;
            }
        }
    }
};

// One position (VEC elements) of all M workers.  `active` is false for the lanes a DIAG warp
// carries past the end of the chunk: they touch no memory and contribute zeros to the sums.
template <int OPT, typename GT, bool POST, int MASK, int VEC, bool DIAG, bool PLAIN = false>
__device__ __forceinline__ void generic_position(const StepArgs &a, char *const (*sp)[GEN_MAX_M],
                                                 const float *sscale, long long e, bool active,
                                                 const WarpDiag<DIAG> &wd) {
    const int M = a.M;
    constexpr bool SX = MASK & SYNC_X, SU = MASK & SYNC_U;
    constexpr bool SV = (OPT != OPT_SGDM) && (MASK & SYNC_V);
    if constexpr (!POST) {
        FV<VEC> xb{}, ub{}, vb{};
        means_of_workers<VEC, SX, SU, SV>(sp, M, e, active, xb, ub, vb);
        constexpr bool NEED_V = OPT != OPT_SGDM && (!SV || OPT == OPT_ADOPT);
                constexpr int B0 = gen_batch(worker_regs<OPT, GT>(!SX, !SU, NEED_V), GEN_BUDGET);
        constexpr int B = (OPT == OPT_ADOPT && B0 > 2) ? 2 : B0;  // ADOPT's normaliser needs more registers
#pragma unroll 1
        for (int m0 = 0; m0 < M; m0 += B) {
            FV<VEC> G[B], X[B], U[B], V[B];
#pragma unroll
            for (int b = 0; b < B; ++b) {
                if (active && m0 + b < M) {
                    G[b] = ld_grad<VEC, GT>(sp[3][m0 + b], e);
                    if constexpr (!SX) X[b] = ld_f32<VEC>(sp[0][m0 + b], e);
                    if constexpr (!SU) U[b] = ld_f32<VEC>(sp[1][m0 + b], e);
                    if constexpr (NEED_V) V[b] = ld_f32<VEC>(sp[2][m0 + b], e);
                }
            }
#pragma unroll
            for (int b = 0; b < B; ++b) {
                if (m0 + b < M) {
                    float gg = 0.f, dd = 0.f, xx = 0.f;
                    if (active) {
                        gg = sum_sq<VEC>(G[b]);
                        const float sc = PLAIN ? 1.f : sscale[m0 + b];
                        FV<VEC> D;
#pragma unroll
                        for (int c = 0; c < VEC; ++c) {
                            const float up = SU ? ub.a[c] : U[b].a[c];
                            const float vown = NEED_V ? V[b].a[c] : 0.f;
                            const float vp = SV ? vb.a[c] : vown;
                            const float xp = SX ? xb.a[c] : X[b].a[c];
                            float un, vn;
                            state_update<OPT, PLAIN>(a, PLAIN ? G[b].a[c] : G[b].a[c] * sc, up, vp, vown, un, vn);
                            D.a[c] = direction<OPT>(a, un, vn);
                            X[b].a[c] = apply_step(a, xp, D.a[c]);
                            U[b].a[c] = un;
                            V[b].a[c] = vn;
                        }
                        dd = sum_sq<VEC>(D);
                        xx = sum_sq<VEC>(X[b]);
                        st_f32<VEC>(sp[0][m0 + b], e, X[b]);
                        st_f32<VEC>(sp[1][m0 + b], e, U[b]);
                        if constexpr (OPT != OPT_SGDM) st_f32<VEC>(sp[2][m0 + b], e, V[b]);
                    }
                    wd.add(DIAG_G, m0 + b, gg);
                    wd.add(DIAG_D, m0 + b, dd);
                    wd.add(DIAG_X, m0 + b, xx);
                }
            }
        }
    } else {
        using P = PostPlan<OPT, MASK>;
        WorkerSum<VEC> au, av, ax;
        au.clear(); av.clear(); ax.clear();
        constexpr int BA = gen_batch(worker_regs<OPT, GT>(!P::D_NEEDS_MEAN, true, OPT != OPT_SGDM), GEN_BUDGET);
        // phase A: states (and x where d_t needs no mean)
#pragma unroll 1
        for (int m0 = 0; m0 < M; m0 += BA) {
            FV<VEC> G[BA], U[BA], V[BA], X[BA];
#pragma unroll
            for (int b = 0; b < BA; ++b) {
                if (active && m0 + b < M) {
                    G[b] = ld_grad<VEC, GT>(sp[3][m0 + b], e);
                    U[b] = ld_f32<VEC>(sp[1][m0 + b], e);
                    if constexpr (OPT != OPT_SGDM) V[b] = ld_f32<VEC>(sp[2][m0 + b], e);
                    if constexpr (!P::D_NEEDS_MEAN) X[b] = ld_f32<VEC>(sp[0][m0 + b], e);
                }
            }
#pragma unroll
            for (int b = 0; b < BA; ++b) {
                if (m0 + b < M) {
                    float gg = 0.f, dd = 0.f, xx = 0.f;
                    if (active) {
                        gg = sum_sq<VEC>(G[b]);
                        const float sc = PLAIN ? 1.f : sscale[m0 + b];
                        FV<VEC> D;
#pragma unroll
                        for (int c = 0; c < VEC; ++c) {
                            const float vown = OPT != OPT_SGDM ? V[b].a[c] : 0.f;
                            float un, vn;
                            state_update<OPT, PLAIN>(a, PLAIN ? G[b].a[c] : G[b].a[c] * sc, U[b].a[c], vown, vown, un, vn);
                            U[b].a[c] = un;
                            V[b].a[c] = vn;
                            if constexpr (!P::D_NEEDS_MEAN) {
                                D.a[c] = direction<OPT>(a, un, vn);
                                X[b].a[c] = apply_step(a, X[b].a[c], D.a[c]);
                            }
                        }
                        // a state that is not averaged has its final value now (phase B re-reads
                        // it where Adam needs it per worker)
                        if constexpr (!P::SU) st_f32<VEC>(sp[1][m0 + b], e, U[b]);
                        if constexpr (OPT != OPT_SGDM && !P::SV) st_f32<VEC>(sp[2][m0 + b], e, V[b]);
                        if constexpr (!P::D_NEEDS_MEAN) {
                            dd = sum_sq<VEC>(D);
                            if constexpr (!P::SX) {
                                xx = sum_sq<VEC>(X[b]);
                                st_f32<VEC>(sp[0][m0 + b], e, X[b]);
                            }
                        }
                    }
                    wd.add(DIAG_G, m0 + b, gg);
                    if constexpr (!P::D_NEEDS_MEAN) {
                        wd.add(DIAG_D, m0 + b, dd);
                        if constexpr (!P::SX) wd.add(DIAG_X, m0 + b, xx);
                    }
                }
            }
            if (active) {
                if constexpr (P::SU) au.template add_batch<BA>(U, M - m0);
                if constexpr (P::SV) av.template add_batch<BA>(V, M - m0);
                if constexpr (P::SX && !P::D_NEEDS_MEAN) ax.template add_batch<BA>(X, M - m0);
            }
        }
        const FV<VEC> mu = au.mean(M), mv = av.mean(M);
        if constexpr (P::D_NEEDS_MEAN) {
            // phase B: parameter step with the averaged states
            constexpr int BB = gen_batch(4 + ((P::KEEP_U || P::KEEP_V) ? 4 : 0), GEN_BUDGET);
#pragma unroll 1
            for (int m0 = 0; m0 < M; m0 += BB) {
                FV<VEC> X[BB], K[BB];
#pragma unroll
                for (int b = 0; b < BB; ++b) {
                    if (active && m0 + b < M) {
                        X[b] = ld_f32<VEC>(sp[0][m0 + b], e);
                        if constexpr (P::KEEP_U) K[b] = ld_f32<VEC>(sp[1][m0 + b], e);
                        if constexpr (P::KEEP_V) K[b] = ld_f32<VEC>(sp[2][m0 + b], e);
                    }
                }
#pragma unroll
                for (int b = 0; b < BB; ++b) {
                    if (m0 + b < M) {
                        float dd = 0.f, xx = 0.f;
                        if (active) {
                            FV<VEC> D;
#pragma unroll
                            for (int c = 0; c < VEC; ++c) {
                                const float un = P::SU ? mu.a[c] : K[b].a[c];
                                const float vn = P::SV ? mv.a[c] : (P::KEEP_V ? K[b].a[c] : 0.f);
                                D.a[c] = direction<OPT>(a, un, vn);
                                X[b].a[c] = apply_step(a, X[b].a[c], D.a[c]);
                            }
                            dd = sum_sq<VEC>(D);
                            if constexpr (!P::SX) {
                                xx = sum_sq<VEC>(X[b]);
                                st_f32<VEC>(sp[0][m0 + b], e, X[b]);
                            }
                            if constexpr (P::SU) st_f32<VEC>(sp[1][m0 + b], e, mu);
                            if constexpr (P::SV) st_f32<VEC>(sp[2][m0 + b], e, mv);
                        }
                        wd.add(DIAG_D, m0 + b, dd);
                        if constexpr (!P::SX) wd.add(DIAG_X, m0 + b, xx);
                    }
                }
                if constexpr (P::SX) {
                    if (active) ax.template add_batch<BB>(X, M - m0);
                }
            }
        }
        if constexpr (P::SX || (!P::D_NEEDS_MEAN && P::SV)) {
            const FV<VEC> mx = ax.mean(M);
            const float xx = (P::SX && active) ? sum_sq<VEC>(mx) : 0.f;
            if (active) {
#pragma unroll 1
                for (int m = 0; m < M; ++m) {
                    if constexpr (P::SX) st_f32<VEC>(sp[0][m], e, mx);
                    if constexpr (!P::D_NEEDS_MEAN && P::SV) st_f32<VEC>(sp[2][m], e, mv);
                }
            }
            if constexpr (P::SX) wd.add_all(DIAG_X, M, xx);
        }
    }
}

template <int OPT, typename GT, bool POST, int MASK, bool DIAG>
__global__ void __launch_bounds__(BLOCK_THREADS, GEN_MIN_BLOCKS)
desloc_step_generic_kernel(const __grid_constant__ StepArgs a) {
    __shared__ char *sp[4][GEN_MAX_M];
    __shared__ float sscale[GEN_MAX_M];
    __shared__ float srows[DIAG ? (BLOCK_THREADS / 32) * DIAG_KINDS * GEN_MAX_M : 1];
    const WarpDiag<DIAG> wd{srows};
    const int tid = threadIdx.x;
    const int lane = tid & 31;
    // exactly one chunk per block (this kernel does not stride: with a chunk loop around the
    // same body the compiler needs spill slots)
    const long long c = blockIdx.x;
    if (c < a.nchunks) {
        const Chunk ch = a.chunks[c];
        int mis = 0;
        for (int m = tid; m < a.M; m += BLOCK_THREADS) {
            const long long idx = static_cast<long long>(m) * a.nt + ch.tensor;
            char *px = reinterpret_cast<char *>(a.x[idx]) + ch.start * 4;
            char *pu = reinterpret_cast<char *>(a.u[idx]) + ch.start * 4;
            char *pv = (OPT != OPT_SGDM) ? reinterpret_cast<char *>(a.v[idx]) + ch.start * 4 : nullptr;
            char *pg = const_cast<char *>(reinterpret_cast<const char *>(grad_ptr(a, idx))) +
                       ch.start * static_cast<long long>(sizeof(GT));
            sp[0][m] = px; sp[1][m] = pu; sp[2][m] = pv; sp[3][m] = pg;
            sscale[m] = a.gscale ? a.gscale[m] : 1.f;
            mis |= (reinterpret_cast<uintptr_t>(px) | reinterpret_cast<uintptr_t>(pu) |
                    reinterpret_cast<uintptr_t>(pv)) & 15u;
            mis |= reinterpret_cast<uintptr_t>(pg) & (sizeof(GT) == 2 ? 7u : 15u);
        }
        if constexpr (DIAG) {
            for (int j = tid; j < (BLOCK_THREADS / 32) * DIAG_KINDS * GEN_MAX_M; j += BLOCK_THREADS)
                srows[j] = 0.f;
        }
        const bool scalar_path = __syncthreads_or(mis) != 0;
        // DIAG warps run whole: lanes past the end take part in the shuffles with zeros
        if (!scalar_path) {
            const int n4 = ch.count >> 2;
            // (no gradient factor and no coordinate clip, the common case: a copy of the loop
            // without them -- this kernel is bound by instruction issue)
            if (a.gscale == nullptr && a.rho > 3.4028235e38f) {
                for (int p = tid; DIAG ? (p - lane < n4) : (p < n4); p += BLOCK_THREADS)
                    generic_position<OPT, GT, POST, MASK, 4, DIAG, true>(a, sp, sscale, static_cast<long long>(p) * 4,
                                                                        p < n4, wd);
            } else {
                for (int p = tid; DIAG ? (p - lane < n4) : (p < n4); p += BLOCK_THREADS)
                    generic_position<OPT, GT, POST, MASK, 4, DIAG>(a, sp, sscale, static_cast<long long>(p) * 4,
                                                                  p < n4, wd);
            }
            const int rem = ch.count & 3;
            if (DIAG ? (tid < 32 && rem > 0) : (tid < rem))
                generic_position<OPT, GT, POST, MASK, 1, DIAG>(a, sp, sscale, (n4 << 2) + tid, tid < rem, wd);
        } else {
            for (int e = tid; DIAG ? (e - lane < ch.count) : (e < ch.count); e += BLOCK_THREADS)
                generic_position<OPT, GT, POST, MASK, 1, DIAG>(a, sp, sscale, e, e < ch.count, wd);
        }
        if constexpr (DIAG) {
            __syncthreads();
            for (int j = tid; j < DIAG_KINDS * a.M; j += BLOCK_THREADS) {
                const int kind = j / a.M, m = j - kind * a.M;
                float total = 0.f;
#pragma unroll
                for (int w = 0; w < BLOCK_THREADS / 32; ++w)
                    total += srows[(w * DIAG_KINDS + kind) * GEN_MAX_M + m];
                a.diag[(static_cast<long long>(kind) * a.M + m) * a.diag_stride + a.diag_chunk0 + c] = total;
            }
        }
    }
}

template <int OPT, typename GT, bool POST, bool DIAG, int MASK>
const void *generic_ptr() {
    return reinterpret_cast<const void *>(&desloc_step_generic_kernel<OPT, GT, POST, MASK, DIAG>);
}

template <int OPT, typename GT, bool POST, bool DIAG>
const void *pick_mask(int mask) {
    switch (mask) {
        case 1: return generic_ptr<OPT, GT, POST, DIAG, 1>();
        case 2: return generic_ptr<OPT, GT, POST, DIAG, 2>();
        case 3: return generic_ptr<OPT, GT, POST, DIAG, 3>();
        default: break;
    }
    if constexpr (OPT != OPT_SGDM) {
        switch (mask) {
            case 4: return generic_ptr<OPT, GT, POST, DIAG, 4>();
            case 5: return generic_ptr<OPT, GT, POST, DIAG, 5>();
            case 6: return generic_ptr<OPT, GT, POST, DIAG, 6>();
            case 7: return generic_ptr<OPT, GT, POST, DIAG, 7>();
            default: break;
        }
    }
    return nullptr;
}

template <int OPT, typename GT>
const void *pick_generic(bool post, int mask, bool diag) {
    if (post) return diag ? pick_mask<OPT, GT, true, true>(mask) : pick_mask<OPT, GT, true, false>(mask);
    return diag ? pick_mask<OPT, GT, false, true>(mask) : pick_mask<OPT, GT, false, false>(mask);
}

}  // namespace

const void *lookup_generic_kernel(int opt, bool post, bool bf16, int mask, bool diag) {
    if (opt == OPT_ADAM)
        return bf16 ? pick_generic<OPT_ADAM, bf16_t>(post, mask, diag) : pick_generic<OPT_ADAM, float>(post, mask, diag);
    if (opt == OPT_ADOPT)
        return bf16 ? pick_generic<OPT_ADOPT, bf16_t>(post, mask, diag) : pick_generic<OPT_ADOPT, float>(post, mask, diag);
    if (opt == OPT_SGDM)
        return bf16 ? pick_generic<OPT_SGDM, bf16_t>(post, mask, diag) : pick_generic<OPT_SGDM, float>(post, mask, diag);
    return nullptr;
}

}  // namespace desloc
