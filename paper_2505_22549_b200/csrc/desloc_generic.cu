// DES-LOC step for worker counts beyond the register-resident kernels (M > MAX_MT) on steps
// that average something.  Same update (update_coord with one worker at a time), runtime M and
// mask.  Worker sums are accumulated in fp64 in the order m = 0..M-1, which is exact for equal
// replicas and matches a sequential reference to rounding.
//
// Pre-average ordering: pass 1 reads only the arrays to be averaged and forms their means;
// pass 2 reads the remaining arrays and updates every worker -- each array is still read once
// (ADOPT re-reads its own v on v-sync steps for the normaliser).  Post-average ordering needs
// the updated states of all workers before any parameter step, so it stores the local u, v
// first and revisits them (the revisit is served from cache).
#include "desloc_kernels.cuh"

namespace desloc {

struct Ptrs {
    char *x, *u, *v;
    const char *g;
};

template <int OPT, typename GT>
__device__ __forceinline__ Ptrs worker_ptrs(const StepArgs &a, const Chunk &ch, int m) {
    const long long idx = static_cast<long long>(m) * a.nt + ch.tensor;
    Ptrs p;
    p.x = reinterpret_cast<char *>(a.x[idx]) + ch.start * 4;
    p.u = reinterpret_cast<char *>(a.u[idx]) + ch.start * 4;
    p.v = (OPT != OPT_SGDM) ? reinterpret_cast<char *>(a.v[idx]) + ch.start * 4 : nullptr;
    p.g = reinterpret_cast<const char *>(grad_ptr(a, idx)) + ch.start * static_cast<long long>(sizeof(GT));
    return p;
}

template <int VEC>
__device__ __forceinline__ void acc_add(double (&acc)[VEC], const FV<VEC> &v) {
#pragma unroll
    for (int c = 0; c < VEC; ++c) acc[c] += static_cast<double>(v.a[c]);
}

template <int VEC>
__device__ __forceinline__ FV<VEC> acc_mean(const double (&acc)[VEC], int M) {
    FV<VEC> r;
#pragma unroll
    for (int c = 0; c < VEC; ++c) r.a[c] = static_cast<float>(acc[c] / static_cast<double>(M));
    return r;
}

// default-cached loads here: the second visit of an address should hit in L1/L2
template <int VEC>
__device__ __forceinline__ FV<VEC> ld_plain(const char *base, long long e) {
    FV<VEC> r;
    if constexpr (VEC == 4) {
        const float4 t = *(reinterpret_cast<const float4 *>(base) + (e >> 2));
        r.a[0] = t.x; r.a[1] = t.y; r.a[2] = t.z; r.a[3] = t.w;
    } else {
        r.a[0] = *(reinterpret_cast<const float *>(base) + e);
    }
    return r;
}

// CMASK >= 0: the sync mask is a compile-time constant (pre-average instantiations, so that
// arrays that are not averaged cost no registers); CMASK < 0: taken from mask_rt.
template <int OPT, typename GT, bool POST, int CMASK, int VEC>
__device__ __forceinline__ void generic_position(const StepArgs &a, const Chunk &ch, int mask_rt,
                                                 long long e) {
    const int mask = CMASK >= 0 ? CMASK : mask_rt;
    const int M = a.M;
    const bool sx = mask & SYNC_X, su = mask & SYNC_U, sv = (OPT != OPT_SGDM) && (mask & SYNC_V);
    if constexpr (!POST) {
        double ax[VEC] = {}, au[VEC] = {}, av[VEC] = {};
        // several workers at a time so that their pointer and data loads overlap (four when one
        // array is averaged, two for two, one for three: more would spill under the register
        // cap); the sums still run in the order m = 0..M-1
        constexpr int NSYNC = CMASK < 0 ? 3 : ((CMASK & 1) + ((CMASK >> 1) & 1) + ((CMASK >> 2) & 1));
        constexpr int NB = NSYNC <= 1 ? 4 : (NSYNC == 2 ? 2 : 1);
#pragma unroll 1
        for (int m0 = 0; m0 < M; m0 += NB) {
            FV<VEC> bx[NB], bu[NB], bv[NB];
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                if (m0 + j < M) {
                    const Ptrs p = worker_ptrs<OPT, GT>(a, ch, m0 + j);
                    if (sx) bx[j] = ld_plain<VEC>(p.x, e);
                    if (su) bu[j] = ld_plain<VEC>(p.u, e);
                    if (sv) bv[j] = ld_plain<VEC>(p.v, e);
                }
            }
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                if (m0 + j < M) {
                    if (sx) acc_add<VEC>(ax, bx[j]);
                    if (su) acc_add<VEC>(au, bu[j]);
                    if (sv) acc_add<VEC>(av, bv[j]);
                }
            }
        }
        const FV<VEC> xb = acc_mean<VEC>(ax, M), ub = acc_mean<VEC>(au, M), vb = acc_mean<VEC>(av, M);
        for (int m = 0; m < M; ++m) {
            const Ptrs p = worker_ptrs<OPT, GT>(a, ch, m);
            FV<VEC> G = ld_grad<VEC, GT>(p.g, e);
            if (a.gscale) {
                const float sc = a.gscale[m];
#pragma unroll
                for (int c = 0; c < VEC; ++c) G.a[c] *= sc;
            }
            FV<VEC> X = sx ? xb : ld_f32<VEC>(p.x, e);
            FV<VEC> U = su ? ub : ld_f32<VEC>(p.u, e);
            FV<VEC> V{}, Vown{};
            if constexpr (OPT != OPT_SGDM) {
                if (OPT == OPT_ADOPT || !sv) Vown = ld_plain<VEC>(p.v, e);
                V = sv ? vb : Vown;
            }
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                // one worker at a time: hand the averaged values in as that worker's "previous"
                // state; ADOPT's normaliser must see the worker's own v, so split it out.
                float g1[1] = {G.a[c]}, x1[1] = {X.a[c]}, u1[1] = {U.a[c]}, v1[1] = {V.a[c]};
                if constexpr (OPT == OPT_ADOPT) {
                    const float gh = fminf(fmaxf(g1[0], -a.rho), a.rho);
                    const float vn = fmaf(a.b2, v1[0], (a.omb2 * gh) * gh);
                    float r = gh / fmaxf(sqrtf(Vown.a[c]), a.eps);
                    r = fminf(fmaxf(r, -a.cbound), a.cbound);
                    const float un = fmaf(a.b1, u1[0], a.omb1 * r);
                    const float d = a.lr * un;
                    x1[0] = x1[0] - fmaf(a.lrwd, x1[0], d);
                    u1[0] = un;
                    v1[0] = vn;
                } else {
                    update_coord<OPT, 0, 1, false>(a, g1, x1, u1, v1);
                }
                X.a[c] = x1[0]; U.a[c] = u1[0]; V.a[c] = v1[0];
            }
            st_f32<VEC>(p.x, e, X);
            st_f32<VEC>(p.u, e, U);
            if constexpr (OPT != OPT_SGDM) st_f32<VEC>(p.v, e, V);
        }
    } else {
        // pass A: local state updates, stored; sums of the ones to be averaged
        double au[VEC] = {}, av[VEC] = {}, ax[VEC] = {};
        for (int m = 0; m < M; ++m) {
            const Ptrs p = worker_ptrs<OPT, GT>(a, ch, m);
            FV<VEC> G = ld_grad<VEC, GT>(p.g, e);
            if (a.gscale) {
                const float sc = a.gscale[m];
#pragma unroll
                for (int c = 0; c < VEC; ++c) G.a[c] *= sc;
            }
            FV<VEC> U = ld_f32<VEC>(p.u, e), V{};
            if constexpr (OPT != OPT_SGDM) V = ld_f32<VEC>(p.v, e);
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                const float gh = fminf(fmaxf(G.a[c], -a.rho), a.rho);
                if constexpr (OPT == OPT_ADAM) {
                    U.a[c] = fmaf(a.b1, U.a[c], a.omb1 * gh);
                    V.a[c] = fmaf(a.b2, V.a[c], (a.omb2 * gh) * gh);
                } else if constexpr (OPT == OPT_ADOPT) {
                    float r = gh / fmaxf(sqrtf(V.a[c]), a.eps);
                    r = fminf(fmaxf(r, -a.cbound), a.cbound);
                    U.a[c] = fmaf(a.b1, U.a[c], a.omb1 * r);
                    V.a[c] = fmaf(a.b2, V.a[c], (a.omb2 * gh) * gh);
                } else {
                    U.a[c] = fmaf(a.b1, U.a[c], a.omb1 * gh);
                }
            }
            if (su) acc_add<VEC>(au, U);
            if (sv) acc_add<VEC>(av, V);
            // plain stores: pass B reads these back
            if constexpr (VEC == 4) {
                *(reinterpret_cast<float4 *>(p.u) + (e >> 2)) = make_float4(U.a[0], U.a[1], U.a[2], U.a[3]);
                if constexpr (OPT != OPT_SGDM)
                    *(reinterpret_cast<float4 *>(p.v) + (e >> 2)) = make_float4(V.a[0], V.a[1], V.a[2], V.a[3]);
            } else {
                *(reinterpret_cast<float *>(p.u) + e) = U.a[0];
                if constexpr (OPT != OPT_SGDM) *(reinterpret_cast<float *>(p.v) + e) = V.a[0];
            }
        }
        const FV<VEC> ub = acc_mean<VEC>(au, M), vb = acc_mean<VEC>(av, M);
        // pass B: parameter step with the (possibly averaged) new states
        for (int m = 0; m < M; ++m) {
            const Ptrs p = worker_ptrs<OPT, GT>(a, ch, m);
            FV<VEC> X = ld_f32<VEC>(p.x, e);
            FV<VEC> U = su ? ub : ld_plain<VEC>(p.u, e), V{};
            if constexpr (OPT == OPT_ADAM) V = sv ? vb : ld_plain<VEC>(p.v, e);
#pragma unroll
            for (int c = 0; c < VEC; ++c) {
                float d;
                if constexpr (OPT == OPT_ADAM)
                    d = (a.lr * U.a[c]) / sqrtf(V.a[c] + a.lam2);
                else
                    d = a.lr * U.a[c];
                X.a[c] = X.a[c] - fmaf(a.lrwd, X.a[c], d);
            }
            if (sx) acc_add<VEC>(ax, X); else st_f32<VEC>(p.x, e, X);
            if (su) st_f32<VEC>(p.u, e, ub);
            if constexpr (OPT != OPT_SGDM) if (sv) st_f32<VEC>(p.v, e, vb);
        }
        if (sx) {
            const FV<VEC> xb = acc_mean<VEC>(ax, M);
            for (int m = 0; m < M; ++m) {
                const Ptrs p = worker_ptrs<OPT, GT>(a, ch, m);
                st_f32<VEC>(p.x, e, xb);
            }
        }
    }
}

template <int OPT, typename GT, bool POST, int CMASK>
__global__ void __launch_bounds__(BLOCK_THREADS, 4)
desloc_step_generic_kernel(const __grid_constant__ StepArgs a, const int mask) {
    __shared__ int s_mis;
    const int tid = threadIdx.x;
    for (long long c = blockIdx.x; c < a.nchunks; c += gridDim.x) {
        const Chunk ch = a.chunks[c];
        if (tid == 0) s_mis = 0;
        __syncthreads();
        // alignment of every worker's four pointers decides vector vs scalar for the chunk
        int mis = 0;
        for (int m = tid; m < a.M; m += BLOCK_THREADS) {
            const Ptrs p = worker_ptrs<OPT, GT>(a, ch, m);
            mis |= (reinterpret_cast<uintptr_t>(p.x) | reinterpret_cast<uintptr_t>(p.u)) & 15u;
            if (OPT != OPT_SGDM) mis |= reinterpret_cast<uintptr_t>(p.v) & 15u;
            mis |= reinterpret_cast<uintptr_t>(p.g) & (sizeof(GT) == 2 ? 7u : 15u);
        }
        if (mis) atomicOr(&s_mis, 1);
        __syncthreads();
        const bool scalar_path = s_mis != 0;
        __syncthreads();
        if (!scalar_path) {
            const int n4 = ch.count >> 2;
            for (int p0 = tid; p0 < n4; p0 += BLOCK_THREADS)
                generic_position<OPT, GT, POST, CMASK, 4>(a, ch, mask, static_cast<long long>(p0) * 4);
            const int rem = ch.count & 3;
            if (tid < rem) generic_position<OPT, GT, POST, CMASK, 1>(a, ch, mask, (n4 << 2) + tid);
        } else {
            for (int e = tid; e < ch.count; e += BLOCK_THREADS)
                generic_position<OPT, GT, POST, CMASK, 1>(a, ch, mask, e);
        }
    }
}

template <int OPT, typename GT, bool POST, int CMASK>
static const void *generic_ptr() {
    return reinterpret_cast<const void *>(&desloc_step_generic_kernel<OPT, GT, POST, CMASK>);
}

template <int OPT, typename GT>
static const void *pick_generic(bool post, int mask) {
    if (post) return generic_ptr<OPT, GT, true, -1>();
    switch (mask) {
        case 1: return generic_ptr<OPT, GT, false, 1>();
        case 2: return generic_ptr<OPT, GT, false, 2>();
        case 3: return generic_ptr<OPT, GT, false, 3>();
        default: break;
    }
    if constexpr (OPT != OPT_SGDM) {
        switch (mask) {
            case 4: return generic_ptr<OPT, GT, false, 4>();
            case 5: return generic_ptr<OPT, GT, false, 5>();
            case 6: return generic_ptr<OPT, GT, false, 6>();
            case 7: return generic_ptr<OPT, GT, false, 7>();
            default: break;
        }
    }
    return nullptr;
}

const void *lookup_generic_kernel(int opt, bool post, bool bf16, int mask) {
    if (opt == OPT_ADAM) return bf16 ? pick_generic<OPT_ADAM, bf16_t>(post, mask) : pick_generic<OPT_ADAM, float>(post, mask);
    if (opt == OPT_ADOPT) return bf16 ? pick_generic<OPT_ADOPT, bf16_t>(post, mask) : pick_generic<OPT_ADOPT, float>(post, mask);
    if (opt == OPT_SGDM) return bf16 ? pick_generic<OPT_SGDM, bf16_t>(post, mask) : pick_generic<OPT_SGDM, float>(post, mask);
    return nullptr;
}

}  // namespace desloc
