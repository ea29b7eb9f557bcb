// desloc_step_static(): one DES-LOC step without a context and without any allocation.
//
// The regular path keeps its chunk table and pointer tables in device memory obtained from
// cudaMalloc at desloc_create().  Some callers cannot do that: a training process whose
// framework has already reserved all of HBM for its own pool (a cudaMalloc then fails, or
// succeeds only by evicting what the pool cached), and loops that must not take the
// device-wide synchronisation cudaMalloc / cudaFree imply.  For them the tables live in a
// fixed array that is part of the library image.
#include <cuda_runtime.h>

#include <cmath>
#include <cstddef>
#include <cstdint>
#include <cstring>
#include <limits>
#include <mutex>

#include "../../include/desloc.h"
#include "desloc_kernels.cuh"

namespace {

constexpr int64_t kMaxPointers = DESLOC_STATIC_MAX_POINTERS;  // M * num_tensors
constexpr int64_t kMaxChunks = DESLOC_STATIC_MAX_CHUNKS;
constexpr int kMaxDevices = 64;

// Layout of the scratch array: [chunks][x table][u table][v table][g table].
struct ScratchImage {
    desloc::Chunk chunks[kMaxChunks];
    void *tables[4][kMaxPointers];
};

// Device-resident scratch, one copy per GPU that loads the library, held until exit.
// In host code this name is only a handle for cudaGetSymbolAddress(); it is not a device
// address and must never be handed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(ScratchImage)];

std::mutex g_setup_mutex;
void *g_scratch_addr[kMaxDevices];  // device address of g_static_scratch per device, once known
bool g_scratch_known[kMaxDevices];

// First call on a device: resolve the device address of the scratch array with that device
// current.  No allocation happens here; the array is part of the loaded module.
cudaError_t scratch_address(int device, void **out) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_known[device]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[device] = p;
        g_scratch_known[device] = true;
    }
    *out = g_scratch_addr[device];
    return cudaSuccess;
}

}  // namespace

extern "C" DESLOC_API int desloc_step_static(const desloc_config *cfg, float *const *x,
                                             float *const *u, float *const *v,
                                             const void *const *grads, int64_t t, float lr_t,
                                             float clip_bound_t, int cuda_device, void *stream,
                                             uint32_t *mask_out) {
    if (!cfg || !cfg->numel || !x || !u || !grads) return DESLOC_E_NULL;
    if (cfg->opt != DESLOC_ADAM && cfg->opt != DESLOC_ADOPT && cfg->opt != DESLOC_SGDM)
        return DESLOC_E_INVALID;
    if (cfg->grad_dtype != DESLOC_F32 && cfg->grad_dtype != DESLOC_BF16) return DESLOC_E_INVALID;
    if (cfg->flags & ~(DESLOC_FLAG_ADOPT_NORM_CLIP | DESLOC_FLAG_POST_AVERAGE)) return DESLOC_E_INVALID;
    if ((cfg->flags & DESLOC_FLAG_ADOPT_NORM_CLIP) && cfg->opt != DESLOC_ADOPT) return DESLOC_E_INVALID;
    if (cfg->opt != DESLOC_SGDM && !v) return DESLOC_E_NULL;
    if (cfg->M < 1 || cfg->M > desloc::MAX_MT) return cfg->M < 1 ? DESLOC_E_RANGE : DESLOC_E_TOO_LARGE;
    if (cfg->num_tensors < 1 || t < 0 || cuda_device < 0 || cuda_device >= kMaxDevices) return DESLOC_E_RANGE;
    if (cfg->Kx < 0 || cfg->Ku < 0 || cfg->Kv < 0) return DESLOC_E_RANGE;
    auto unit = [](float b) { return std::isfinite(b) && b >= 0.f && b < 1.f; };
    if (!unit(cfg->beta1) || (cfg->opt != DESLOC_SGDM && !unit(cfg->beta2))) return DESLOC_E_RANGE;
    if (!(cfg->eps >= 0.f) || !std::isfinite(cfg->eps)) return DESLOC_E_RANGE;
    if (!(cfg->weight_decay >= 0.f) || !std::isfinite(cfg->weight_decay)) return DESLOC_E_RANGE;
    if (std::isnan(cfg->clip_rho) || !std::isfinite(lr_t)) return DESLOC_E_RANGE;
    const bool nclip = (cfg->flags & DESLOC_FLAG_ADOPT_NORM_CLIP) != 0;
    if (nclip && !(clip_bound_t >= 0.f)) return DESLOC_E_RANGE;

    const int64_t nptr = static_cast<int64_t>(cfg->M) * cfg->num_tensors;
    if (nptr > kMaxPointers) return DESLOC_E_TOO_LARGE;
    int64_t nchunks = 0;
    for (int32_t k = 0; k < cfg->num_tensors; ++k) {
        if (cfg->numel[k] < 1) return DESLOC_E_RANGE;
        nchunks += (cfg->numel[k] + desloc::CHUNK_ELEMS - 1) / desloc::CHUNK_ELEMS;
        if (nchunks > kMaxChunks) return DESLOC_E_TOO_LARGE;
    }
    for (int64_t i = 0; i < nptr; ++i) {
        if (!x[i] || !u[i] || !grads[i]) return DESLOC_E_NULL;
        if (cfg->opt != DESLOC_SGDM && !v[i]) return DESLOC_E_NULL;
    }

    uint32_t mask = desloc_sync_mask(cfg, t);
    const uint32_t kmask = (cfg->M == 1) ? 0u : mask;
    const void *fn = desloc::lookup_step_kernel(cfg->opt, (cfg->flags & DESLOC_FLAG_POST_AVERAGE) != 0,
                                                cfg->grad_dtype == DESLOC_BF16, cfg->M,
                                                static_cast<int>(kmask));
    if (!fn) return DESLOC_E_INVALID;

    // Host image of the tables, on this thread's stack (about 320 KB): no heap, no pinned memory.
    ScratchImage img;
    int64_t c = 0;
    for (int32_t k = 0; k < cfg->num_tensors; ++k)
        for (int64_t s = 0; s < cfg->numel[k]; s += desloc::CHUNK_ELEMS) {
            const int64_t left = cfg->numel[k] - s;
            img.chunks[c].tensor = k;
            img.chunks[c].count = static_cast<int32_t>(left < desloc::CHUNK_ELEMS ? left : desloc::CHUNK_ELEMS);
            img.chunks[c].start = s;
            ++c;
        }
    for (int64_t i = 0; i < nptr; ++i) {
        img.tables[0][i] = x[i];
        img.tables[1][i] = u[i];
        img.tables[2][i] = v ? static_cast<void *>(v[i]) : nullptr;
        img.tables[3][i] = const_cast<void *>(grads[i]);
    }

    int dev_before = -1;
    cudaError_t e = cudaGetDevice(&dev_before);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return DESLOC_E_CUDA; }
    if (dev_before != cuda_device) {
        e = cudaSetDevice(cuda_device);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return DESLOC_E_CUDA; }
    }
    int rc = DESLOC_OK;
    do {
        void *scratch = nullptr;
        e = scratch_address(cuda_device, &scratch);
        if (e != cudaSuccess) { rc = DESLOC_E_CUDA; break; }
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        unsigned char *base = static_cast<unsigned char *>(scratch);
        // Only the parts this call uses are rewritten; nothing in the array has to start at
        // zero.  The copies are ordered before the kernel on `st`.
        e = cudaMemcpyAsync(base + offsetof(ScratchImage, chunks), img.chunks,
                            static_cast<size_t>(nchunks) * sizeof(desloc::Chunk),
                            cudaMemcpyHostToDevice, st);
        for (int a = 0; a < 4 && e == cudaSuccess; ++a)
            e = cudaMemcpyAsync(base + offsetof(ScratchImage, tables) +
                                    static_cast<size_t>(a) * kMaxPointers * sizeof(void *),
                                img.tables[a], static_cast<size_t>(nptr) * sizeof(void *),
                                cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) { rc = DESLOC_E_CUDA; break; }

        desloc::StepArgs a{};
        void **tab = reinterpret_cast<void **>(base + offsetof(ScratchImage, tables));
        a.chunks = reinterpret_cast<const desloc::Chunk *>(base + offsetof(ScratchImage, chunks));
        a.nchunks = nchunks;
        a.x = reinterpret_cast<float *const *>(tab);
        a.u = reinterpret_cast<float *const *>(tab + kMaxPointers);
        a.v = reinterpret_cast<float *const *>(tab + 2 * kMaxPointers);
        a.g = reinterpret_cast<const void *const *>(tab + 3 * kMaxPointers);
        a.gscale = nullptr;
        a.nt = cfg->num_tensors;
        a.M = cfg->M;
        a.b1 = cfg->beta1;
        a.omb1 = static_cast<float>(1.0 - static_cast<double>(cfg->beta1));
        a.b2 = cfg->beta2;
        a.omb2 = static_cast<float>(1.0 - static_cast<double>(cfg->beta2));
        a.eps = cfg->eps;
        a.lam2 = static_cast<float>(static_cast<double>(cfg->eps) * static_cast<double>(cfg->eps));
        a.lr = lr_t;
        a.lrwd = static_cast<float>(static_cast<double>(lr_t) * static_cast<double>(cfg->weight_decay));
        a.rho = cfg->clip_rho > 0.f ? cfg->clip_rho : std::numeric_limits<float>::infinity();
        a.cbound = nclip ? clip_bound_t : std::numeric_limits<float>::infinity();
        const long long nitems =
            (cfg->M == 1) ? (nchunks + desloc::LOCAL_SLOTS - 1) / desloc::LOCAL_SLOTS : nchunks;
        void *params[] = {&a};
        e = cudaLaunchKernel(fn, dim3(static_cast<unsigned>(nitems)), dim3(desloc::BLOCK_THREADS),
                             params, 0, st);
        if (e != cudaSuccess) { rc = DESLOC_E_CUDA; break; }
    } while (false);
    if (rc == DESLOC_E_CUDA) (void)cudaGetLastError();
    if (dev_before != cuda_device) cudaSetDevice(dev_before);
    if (rc == DESLOC_OK && mask_out) *mask_out = mask;
    return rc;
}
