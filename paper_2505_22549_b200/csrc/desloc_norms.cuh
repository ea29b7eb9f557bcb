// Launchers of the reduction kernels (gradient norms, relative state change).
#pragma once
#include "desloc_kernels.cuh"

namespace desloc {

// partial: scratch of at least M * nchunks floats; norms, scales: [M] floats, all on the device.
// scales[m] = min(1, max_norm / ||g^m||_2), or 1 when max_norm <= 0.  Two launches.
// err, wait_limit: the flag a block sets when its bounded wait for a bulk copy runs out, and the
// bound (as for the step kernels).
cudaError_t launch_grad_norms(const Chunk *chunks, long long nchunks, const void *const *g, int nt,
                              int M, bool bf16, float max_norm, float *partial, float *norms,
                              float *scales, int *err, int wait_limit, cudaStream_t stream);

// partial: scratch of at least 2 * M * nchunks floats; out[m] = ||now - then|| / ||then||.
cudaError_t launch_rel_change(const Chunk *chunks, long long nchunks, const float *const *now,
                              const float *const *then, int nt, int M, float *partial, float *out,
                              cudaStream_t stream);

// Norms of a diagnostics step: partial [DIAG_KINDS][M][stride] per-chunk sums of squares,
// tstart [nt + 1] first chunk of every tensor; writes sums [DIAG_KINDS][M][nt] (fp64 scratch),
// per_tensor [DIAG_KINDS][M][nt] and totals [DIAG_KINDS][M] (floats), all on the device.
cudaError_t launch_diag_norms(const float *partial, long long stride, const long long *tstart,
                              int nt, int M, double *sums, float *per_tensor, float *totals,
                              cudaStream_t stream);

// Every element of the m_dst destination replicas := mean over the m_src source replicas.
// src / dst are device tables indexed [m * nt + tensor].
cudaError_t launch_mean_fill(const Chunk *chunks, long long nchunks, const float *const *src,
                             int m_src, float *const *dst, int m_dst, int nt, cudaStream_t stream);

}  // namespace desloc
