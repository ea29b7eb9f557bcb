// Reductions around the DES-LOC step: per-worker gradient norms for norm-based clipping (the
// clipping the paper's language-model runs used), the relative rate of change of a state,
// ||s_now - s_then||_2 / ||s_then||_2 (Section 5.1, "Metrics"), and the finalisation of the
// per-tensor gradient / parameter / update norms a diagnostics step accumulated.
//
// Both are two-stage and deterministic: stage 1 writes one fp32 partial per (worker, chunk)
// -- per-thread sums of up to 16 squares, a shuffle tree, then the eight warp sums in order;
// stage 2 adds the partials of a worker in fp64 in a fixed pattern.  No atomics.
#include "desloc_norms.cuh"

namespace desloc {

namespace {

__device__ __forceinline__ float block_sum(float v, float *warp_sums) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_down_sync(0xffffffffu, v, off);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();  // warp_sums may still be read from the previous use
    if (lane == 0) warp_sums[warp] = v;
    __syncthreads();
    float t = 0.f;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < BLOCK_THREADS / 32; ++w) t += warp_sums[w];
    }
    return t;  // valid in thread 0
}

// partial[m * ngroups + q] = sum of g^m squared over chunk group q (SUMSQ_GROUP consecutive
// chunks).  Work item = (worker, group): a block streams up to 64 KB of one worker's gradient
// with eight independent loads per thread in flight, and reduces once.
constexpr int SUMSQ_GROUP = 8;

template <typename GT>
__device__ __forceinline__ float chunk_sumsq(const Chunk &ch, const void *const *g, int nt, int m,
                                             float acc) {
    const int tid = threadIdx.x;
    const char *base = reinterpret_cast<const char *>(g[static_cast<long long>(m) * nt + ch.tensor]) +
                       ch.start * static_cast<long long>(sizeof(GT));
    const bool aligned = (reinterpret_cast<uintptr_t>(base) & (sizeof(GT) == 2 ? 7u : 15u)) == 0;
    if (aligned) {
        const int n4 = ch.count >> 2;
        FV<4> v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int p = tid + j * BLOCK_THREADS;
            if (p < n4) v[j] = ld_grad<4, GT>(base, static_cast<long long>(p) * 4);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int p = tid + j * BLOCK_THREADS;
            if (p < n4) {
#pragma unroll
                for (int k = 0; k < 4; ++k) acc = fmaf(v[j].a[k], v[j].a[k], acc);
            }
        }
        const int rem = ch.count & 3;
        if (tid < rem) {
            const float t = ld_grad<1, GT>(base, (n4 << 2) + tid).a[0];
            acc = fmaf(t, t, acc);
        }
    } else {
        for (int e = tid; e < ch.count; e += BLOCK_THREADS) {
            const float t = ld_grad<1, GT>(base, e).a[0];
            acc = fmaf(t, t, acc);
        }
    }
    return acc;
}

// Eight bf16 values in one 128-bit load.
__device__ __forceinline__ float sumsq8_bf16(const uint4 &t, float acc) {
    const unsigned w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const float lo = __uint_as_float(w[k] << 16), hi = __uint_as_float(w[k] & 0xffff0000u);
        acc = fmaf(lo, lo, acc);
        acc = fmaf(hi, hi, acc);
    }
    return acc;
}

template <typename GT>
__global__ void __launch_bounds__(BLOCK_THREADS, 3)
sumsq_kernel(const Chunk *chunks, long long nchunks, const void *const *g, int nt, int M,
             float *partial) {
    __shared__ float warp_sums[BLOCK_THREADS / 32];
    const long long ngroups = (nchunks + SUMSQ_GROUP - 1) / SUMSQ_GROUP;
    const long long nitems = ngroups * M;
    const int tid = threadIdx.x;
    for (long long item = blockIdx.x; item < nitems; item += gridDim.x) {
        const long long q = item % ngroups;
        const int m = static_cast<int>(item / ngroups);
        const long long c0 = q * SUMSQ_GROUP;
        float acc0 = 0.f, acc1 = 0.f;
        {
            // All chunk descriptors and gradient pointers of the group first (one dependent-load
            // chain for the whole item), then the data: full, 16-byte aligned chunks take 128-bit
            // loads, eight of them in flight per thread (four bf16 chunks or two fp32 chunks).
            constexpr int LPC = sizeof(GT) == 2 ? 2 : 4;  // 128-bit loads per thread and chunk
            constexpr int CB = 8 / LPC;                   // chunks per batch
            const uint4 *wide[SUMSQ_GROUP];
#pragma unroll
            for (int j = 0; j < SUMSQ_GROUP; ++j) {
                wide[j] = nullptr;
                if (c0 + j < nchunks) {
                    const Chunk ch = chunks[c0 + j];
                    const char *base =
                        reinterpret_cast<const char *>(g[static_cast<long long>(m) * nt + ch.tensor]) +
                        ch.start * static_cast<long long>(sizeof(GT));
                    if (ch.count == REDUCE_CHUNK_ELEMS && (reinterpret_cast<uintptr_t>(base) & 15u) == 0)
                        wide[j] = reinterpret_cast<const uint4 *>(base);
                }
            }
#pragma unroll
            for (int k = 0; k < SUMSQ_GROUP; k += CB) {
                uint4 r[CB][LPC];
#pragma unroll
                for (int j = 0; j < CB; ++j) {
                    if (wide[k + j]) {
#pragma unroll
                        for (int l = 0; l < LPC; ++l)
                            r[j][l] = *(wide[k + j] + tid + l * BLOCK_THREADS);
                    }
                }
#pragma unroll
                for (int j = 0; j < CB; ++j) {
                    if (wide[k + j]) {
#pragma unroll
                        for (int l = 0; l < LPC; ++l) {
                            float &acc = (l & 1) ? acc1 : acc0;
                            if constexpr (sizeof(GT) == 2) {
                                acc = sumsq8_bf16(r[j][l], acc);
                            } else {
                                const float f[4] = {__uint_as_float(r[j][l].x), __uint_as_float(r[j][l].y),
                                                    __uint_as_float(r[j][l].z), __uint_as_float(r[j][l].w)};
#pragma unroll
                                for (int q4 = 0; q4 < 4; ++q4) acc = fmaf(f[q4], f[q4], acc);
                            }
                        }
                    } else if (c0 + k + j < nchunks) {
                        acc0 = chunk_sumsq<GT>(chunks[c0 + k + j], g, nt, m, acc0);
                    }
                }
            }
        }
        const float total = block_sum(acc0 + acc1, warp_sums);
        if (tid == 0) partial[static_cast<long long>(m) * ngroups + q] = total;
    }
}

// The same reduction for bf16 gradients with the group's full, 16-byte aligned chunks brought
// into shared memory by bulk asynchronous copies (8 KB each, all requested at once, three blocks
// per SM: up to 192 KB in flight per SM) and summed from there in the order sumsq_kernel uses,
// so that both kernels give the same bits.  Chunks that cannot be staged are read directly.
// On the 1.7 G-parameter workload (13.7 GB of gradients) the norm-clipped step takes 28.25 ms
// with this pass against 28.45 ms with sumsq_kernel (2.0 ms against 2.2 ms for the pass).
__global__ void __launch_bounds__(BLOCK_THREADS, 3)
sumsq_bulk_kernel(const Chunk *chunks, long long nchunks, const void *const *g, int nt, int M,
                  float *partial, int *err, int wait_limit) {
    using GT = bf16_t;
    constexpr int CHUNK_BYTES = REDUCE_CHUNK_ELEMS * static_cast<int>(sizeof(GT));
    constexpr int LPC = 2, CB = 8 / LPC;   // as in sumsq_kernel
    extern __shared__ __align__(128) char stage[];   // SUMSQ_GROUP chunks
    __shared__ float warp_sums[BLOCK_THREADS / 32];
    __shared__ int s_staged[SUMSQ_GROUP];
    __shared__ __align__(8) uint64_t bar;
    const long long ngroups = (nchunks + SUMSQ_GROUP - 1) / SUMSQ_GROUP;
    const long long nitems = ngroups * M;
    const int tid = threadIdx.x;
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&bar)), "r"(SUMSQ_GROUP) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    uint32_t phase = 0;
    for (long long item = blockIdx.x; item < nitems; item += gridDim.x) {
        const long long q = item % ngroups;
        const int m = static_cast<int>(item / ngroups);
        const long long c0 = q * SUMSQ_GROUP;
        __syncthreads();   // the previous item is done with the stage; the barrier exists
        if (tid < SUMSQ_GROUP) {
            // one thread per chunk of the group: request it, or leave it to the direct path
            uint32_t bytes = 0;
            if (c0 + tid < nchunks) {
                const Chunk ch = chunks[c0 + tid];
                const char *base =
                    reinterpret_cast<const char *>(g[static_cast<long long>(m) * nt + ch.tensor]) +
                    ch.start * static_cast<long long>(sizeof(GT));
                if (ch.count == REDUCE_CHUNK_ELEMS && (reinterpret_cast<uintptr_t>(base) & 15u) == 0) {
                    bytes = CHUNK_BYTES;
                    bulk_load(stage + tid * CHUNK_BYTES, base, bytes, &bar);
                }
            }
            s_staged[tid] = bytes != 0;
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                         :: "r"(smem_u32(&bar)), "r"(bytes) : "memory");
        }
        __syncthreads();
        const bool landed = bar_wait(&bar, phase, wait_limit);
        if (__syncthreads_or(!landed)) {
            // give up: say so, let the copies land (bounded as well), leave
            if (tid == 0 && err) *reinterpret_cast<volatile int *>(err) = 1;
            bar_wait(&bar, phase, DRAIN_WAIT_LIMIT);
            __syncthreads();
            return;
        }
        phase ^= 1u;
        float acc0 = 0.f, acc1 = 0.f;
#pragma unroll
        for (int k = 0; k < SUMSQ_GROUP; k += CB) {
            uint4 r[CB][LPC];
#pragma unroll
            for (int j = 0; j < CB; ++j) {
                if (s_staged[k + j]) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(stage + (k + j) * CHUNK_BYTES);
#pragma unroll
                    for (int l = 0; l < LPC; ++l) r[j][l] = src[tid + l * BLOCK_THREADS];
                }
            }
#pragma unroll
            for (int j = 0; j < CB; ++j) {
                if (s_staged[k + j]) {
#pragma unroll
                    for (int l = 0; l < LPC; ++l) {
                        float &acc = (l & 1) ? acc1 : acc0;
                        acc = sumsq8_bf16(r[j][l], acc);
                    }
                } else if (c0 + k + j < nchunks) {
                    acc0 = chunk_sumsq<GT>(chunks[c0 + k + j], g, nt, m, acc0);
                }
            }
        }
        const float total = block_sum(acc0 + acc1, warp_sums);
        if (tid == 0) partial[static_cast<long long>(m) * ngroups + q] = total;
    }
}

// partial[(0|1) * M * nchunks + m * nchunks + c]: sum of (now - then)^2 and of then^2.
__global__ void __launch_bounds__(BLOCK_THREADS, 6)
relchange_kernel(const Chunk *chunks, long long nchunks, const float *const *now,
                 const float *const *then, int nt, int M, float *partial) {
    __shared__ float warp_sums[BLOCK_THREADS / 32];
    const long long nitems = nchunks * M;
    const int tid = threadIdx.x;
    for (long long item = blockIdx.x; item < nitems; item += gridDim.x) {
        const long long c = item % nchunks;
        const int m = static_cast<int>(item / nchunks);
        const Chunk ch = chunks[c];
        const long long idx = static_cast<long long>(m) * nt + ch.tensor;
        const char *pa = reinterpret_cast<const char *>(now[idx]) + ch.start * 4;
        const char *pb = reinterpret_cast<const char *>(then[idx]) + ch.start * 4;
        const bool aligned = ((reinterpret_cast<uintptr_t>(pa) | reinterpret_cast<uintptr_t>(pb)) & 15u) == 0;
        float num = 0.f, den = 0.f;
        if (aligned) {
            const int n4 = ch.count >> 2;
            for (int p = tid; p < n4; p += BLOCK_THREADS) {
                const FV<4> a = ld_f32<4>(pa, static_cast<long long>(p) * 4);
                const FV<4> b = ld_f32<4>(pb, static_cast<long long>(p) * 4);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float d = a.a[k] - b.a[k];
                    num = fmaf(d, d, num);
                    den = fmaf(b.a[k], b.a[k], den);
                }
            }
            const int rem = ch.count & 3;
            if (tid < rem) {
                const float a = ld_f32<1>(pa, (n4 << 2) + tid).a[0], b = ld_f32<1>(pb, (n4 << 2) + tid).a[0];
                num = fmaf(a - b, a - b, num);
                den = fmaf(b, b, den);
            }
        } else {
            for (int e = tid; e < ch.count; e += BLOCK_THREADS) {
                const float a = ld_f32<1>(pa, e).a[0], b = ld_f32<1>(pb, e).a[0];
                num = fmaf(a - b, a - b, num);
                den = fmaf(b, b, den);
            }
        }
        const float tn = block_sum(num, warp_sums);
        const float td = block_sum(den, warp_sums);
        if (tid == 0) {
            partial[static_cast<long long>(m) * nchunks + c] = tn;
            partial[(static_cast<long long>(M) + m) * nchunks + c] = td;
        }
    }
}

// One block per row: out_sum[row] = sum of partial[row * n .. +n) in fp64, fixed pattern
// (thread i adds entries i, i+256, ... in order; then a shared-memory tree).
template <typename T>
__device__ __forceinline__ double row_sum_f64(const T *row, long long n, double *sh) {
    double acc = 0.0;
    for (long long i = threadIdx.x; i < n; i += BLOCK_THREADS) acc += static_cast<double>(row[i]);
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int s = BLOCK_THREADS / 2; s > 0; s >>= 1) {
        if (threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
        __syncthreads();
    }
    const double r = sh[0];
    __syncthreads();
    return r;
}

// norms[m] = ||g^m||_2, scales[m] = min(1, max_norm / norms[m]) (1 when max_norm <= 0).
__global__ void __launch_bounds__(BLOCK_THREADS)
norm_finalize_kernel(const float *partial, long long nchunks, float max_norm, float *norms,
                     float *scales) {
    __shared__ double sh[BLOCK_THREADS];
    const int m = blockIdx.x;
    const double ss = row_sum_f64(partial + static_cast<long long>(m) * nchunks, nchunks, sh);
    if (threadIdx.x == 0) {
        const double nrm = sqrt(ss);
        norms[m] = static_cast<float>(nrm);
        scales[m] = (max_norm > 0.f && nrm > static_cast<double>(max_norm))
                        ? static_cast<float>(static_cast<double>(max_norm) / nrm)
                        : 1.f;
    }
}

__global__ void __launch_bounds__(BLOCK_THREADS)
relchange_finalize_kernel(const float *partial, long long nchunks, int M, float *out) {
    __shared__ double sh[BLOCK_THREADS];
    const int m = blockIdx.x;
    const double num = row_sum_f64(partial + static_cast<long long>(m) * nchunks, nchunks, sh);
    const double den = row_sum_f64(partial + (static_cast<long long>(M) + m) * nchunks, nchunks, sh);
    if (threadIdx.x == 0) out[m] = static_cast<float>(sqrt(num) / sqrt(den));
}

// dst^j[i] = mean over the M_src source replicas of src^m[i] (fp64 sum in the order
// m = 0..M_src-1, rounded once), for every destination replica j.  Work item = chunk.
__global__ void __launch_bounds__(BLOCK_THREADS, 4)
mean_fill_kernel(const Chunk *chunks, long long nchunks, const float *const *src, int m_src,
                 float *const *dst, int m_dst, int nt) {
    for (long long c = blockIdx.x; c < nchunks; c += gridDim.x) {
        const Chunk ch = chunks[c];
        for (int e = threadIdx.x; e < ch.count; e += BLOCK_THREADS) {
            double acc = 0.0;
            for (int m = 0; m < m_src; ++m)
                acc += static_cast<double>(src[static_cast<long long>(m) * nt + ch.tensor][ch.start + e]);
            const float mean = static_cast<float>(acc / static_cast<double>(m_src));
            for (int j = 0; j < m_dst; ++j)
                dst[static_cast<long long>(j) * nt + ch.tensor][ch.start + e] = mean;
        }
    }
}

// Norm diagnostics of a DIAG step.  partial[(kind * M + m) * stride + c] holds the sum of
// squares of chunk c; tstart[k] .. tstart[k + 1] are the chunks of tensor k.  One block per
// (tensor, worker, kind): fp64 sum of the tensor's chunks, its root as the per-tensor norm.
__global__ void __launch_bounds__(BLOCK_THREADS)
diag_tensor_kernel(const float *partial, long long stride, const long long *tstart, int nt, int M,
                   double *sums, float *norms) {
    __shared__ double sh[BLOCK_THREADS];
    const int k = blockIdx.x, m = blockIdx.y, kind = blockIdx.z;
    const long long row = static_cast<long long>(kind) * M + m;
    const double ss = row_sum_f64(partial + row * stride + tstart[k], tstart[k + 1] - tstart[k], sh);
    if (threadIdx.x == 0) {
        sums[row * nt + k] = ss;
        norms[row * nt + k] = static_cast<float>(sqrt(ss));
    }
}

// One block per (kind, worker): the whole-model norm from the per-tensor sums of squares.
__global__ void __launch_bounds__(BLOCK_THREADS)
diag_total_kernel(const double *sums, int nt, float *totals) {
    __shared__ double sh[BLOCK_THREADS];
    const long long row = blockIdx.x;
    const double ss = row_sum_f64(sums + row * nt, nt, sh);
    if (threadIdx.x == 0) totals[row] = static_cast<float>(sqrt(ss));
}

unsigned grid_for(long long nitems) {
    return static_cast<unsigned>(nitems < 0x7fffffffLL ? (nitems > 0 ? nitems : 1) : 0x7fffffffLL);
}

}  // namespace

cudaError_t launch_grad_norms(const Chunk *chunks, long long nchunks, const void *const *g, int nt,
                              int M, bool bf16, float max_norm, float *partial, float *norms,
                              float *scales, int *err, int wait_limit, cudaStream_t stream) {
    const long long ngroups = (nchunks + SUMSQ_GROUP - 1) / SUMSQ_GROUP;
    const unsigned grid = grid_for(ngroups * M);
    if (bf16) {
        constexpr int smem = SUMSQ_GROUP * REDUCE_CHUNK_ELEMS * 2;
        cudaError_t e0 = cudaFuncSetAttribute(sumsq_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e0 != cudaSuccess) return e0;
        sumsq_bulk_kernel<<<grid, BLOCK_THREADS, smem, stream>>>(chunks, nchunks, g, nt, M, partial, err,
                                                                 wait_limit);
    } else
        sumsq_kernel<float><<<grid, BLOCK_THREADS, 0, stream>>>(chunks, nchunks, g, nt, M, partial);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    norm_finalize_kernel<<<M, BLOCK_THREADS, 0, stream>>>(partial, ngroups, max_norm, norms, scales);
    return cudaGetLastError();
}

cudaError_t launch_rel_change(const Chunk *chunks, long long nchunks, const float *const *now,
                              const float *const *then, int nt, int M, float *partial, float *out,
                              cudaStream_t stream) {
    relchange_kernel<<<grid_for(nchunks * M), BLOCK_THREADS, 0, stream>>>(chunks, nchunks, now, then,
                                                                          nt, M, partial);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    relchange_finalize_kernel<<<M, BLOCK_THREADS, 0, stream>>>(partial, nchunks, M, out);
    return cudaGetLastError();
}

cudaError_t launch_diag_norms(const float *partial, long long stride, const long long *tstart,
                              int nt, int M, double *sums, float *per_tensor, float *totals,
                              cudaStream_t stream) {
    diag_tensor_kernel<<<dim3(nt, M, DIAG_KINDS), BLOCK_THREADS, 0, stream>>>(partial, stride, tstart,
                                                                            nt, M, sums, per_tensor);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    diag_total_kernel<<<DIAG_KINDS * M, BLOCK_THREADS, 0, stream>>>(sums, nt, totals);
    return cudaGetLastError();
}

cudaError_t launch_mean_fill(const Chunk *chunks, long long nchunks, const float *const *src,
                             int m_src, float *const *dst, int m_dst, int nt, cudaStream_t stream) {
    mean_fill_kernel<<<grid_for(nchunks), BLOCK_THREADS, 0, stream>>>(chunks, nchunks, src, m_src,
                                                                      dst, m_dst, nt);
    return cudaGetLastError();
}

}  // namespace desloc
