// desloc_step_static(): one DES-LOC step without a context and without any allocation.
//
// The regular path keeps its chunk table and pointer tables in device memory obtained from
// cudaMalloc at desloc_create().  Some callers cannot do that: a training process whose
// framework has already reserved all of HBM for its own pool (a cudaMalloc then fails, or
// succeeds only by evicting what the pool cached), and loops that must not take the
// device-wide synchronisation cudaMalloc / cudaFree imply.  For them the tables live in a
// fixed array that is part of the library image.
//
// Validation, the chunk plan and the choice of kernel are the context path's own
// (desloc_internal.cuh), so both paths launch the same grid of the same kernel.
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>
#include <cstring>
#include <mutex>

#include "desloc_internal.cuh"

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

std::mutex g_mutex;                 // guards everything below
void *g_scratch_addr[kMaxDevices];  // device address of g_static_scratch per device, once known
bool g_scratch_known[kMaxDevices];

// Host copy of what the scratch array of device g_mirror_device holds (after the copies this
// library has enqueued there).  A call whose tensor list or pointers equal the mirror's skips
// that upload: a loop that steps the same buffers again and again enqueues no copy at all
// after its first call, and so never waits on the stream.  Static storage, not the heap and
// not the caller's stack.
ScratchImage g_mirror;
int g_mirror_device = -1;
int32_t g_mirror_nt = 0;
int64_t g_mirror_nptr = 0;
int64_t g_mirror_chunk_elems = 0;
int64_t g_mirror_numel[kMaxPointers];
int64_t g_mirror_heads[kMaxPointers];  // short first chunk per tensor of the mirrored plan
int64_t g_heads[kMaxPointers];         // the same for the call in progress

// First call on a device: resolve the device address of the scratch array with that device
// current.  No cudaMalloc happens here; the array is part of the module the runtime loads.
cudaError_t scratch_address(int device, void **out) {
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
    desloc::NvtxRange range("desloc_step_static");
    // ---- everything that can be rejected without touching CUDA ------------------------------
    int rc = desloc::validate_config(cfg);
    if (rc != DESLOC_OK) return rc;
    if (!x || !u || !grads) return DESLOC_E_NULL;
    if (cfg->opt != DESLOC_SGDM && !v) return DESLOC_E_NULL;
    rc = desloc::validate_numel(cfg, nullptr);
    if (rc != DESLOC_OK) return rc;
    if (t < 0 || cuda_device < 0 || cuda_device >= kMaxDevices) return DESLOC_E_RANGE;
    rc = desloc::validate_step(cfg, lr_t, clip_bound_t);
    if (rc != DESLOC_OK) return rc;
    if (cfg->M > desloc::MAX_MT) return DESLOC_E_TOO_LARGE;
    const int64_t nptr = static_cast<int64_t>(cfg->M) * cfg->num_tensors;
    if (nptr > kMaxPointers) return DESLOC_E_TOO_LARGE;
    for (int64_t i = 0; i < nptr; ++i) {
        if (!x[i] || !u[i] || !grads[i]) return DESLOC_E_NULL;
        if (cfg->opt != DESLOC_SGDM && !v[i]) return DESLOC_E_NULL;
    }
    std::lock_guard<std::mutex> lock(g_mutex);
    const int64_t chunk_elems = desloc::chunk_elems_for(cfg->M, cfg->numel, cfg->num_tensors);
    for (int32_t k = 0; k < cfg->num_tensors; ++k) g_heads[k] = desloc::head_elems(x[k], cfg->numel[k]);
    const int64_t nchunks = desloc::count_chunks(cfg->numel, cfg->num_tensors, chunk_elems, g_heads);
    if (nchunks > kMaxChunks) return DESLOC_E_TOO_LARGE;
    const uint32_t mask = desloc::mask_at(cfg, t);
    const desloc::LaunchPlan plan = desloc::plan_launch(*cfg, mask, nchunks, false);
    if (!plan.fn) return DESLOC_E_INVALID;

    int dev_before = -1;
    cudaError_t e = cudaGetDevice(&dev_before);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return DESLOC_E_CUDA; }
    if (dev_before != cuda_device) {
        e = cudaSetDevice(cuda_device);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return DESLOC_E_CUDA; }
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    do {
        // The uploads below read host memory this library reuses on the next call: a captured
        // copy would replay whatever that memory holds by then.  Refuse, capturing nothing.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        e = cudaStreamIsCapturing(st, &cap);
        if (e != cudaSuccess) { rc = DESLOC_E_CUDA; break; }
        if (cap != cudaStreamCaptureStatusNone) { rc = DESLOC_E_INVALID; break; }

        void *scratch = nullptr;
        e = scratch_address(cuda_device, &scratch);
        if (e != cudaSuccess) { rc = DESLOC_E_CUDA; break; }
        unsigned char *base = static_cast<unsigned char *>(scratch);

        // What of the mirror still describes this device's array?
        const bool same_device = g_mirror_device == cuda_device;
        const bool same_plan = same_device && g_mirror_nt == cfg->num_tensors &&
                               g_mirror_chunk_elems == chunk_elems &&
                               std::memcmp(g_mirror_numel, cfg->numel,
                                           static_cast<size_t>(cfg->num_tensors) * sizeof(int64_t)) == 0 &&
                               std::memcmp(g_mirror_heads, g_heads,
                                           static_cast<size_t>(cfg->num_tensors) * sizeof(int64_t)) == 0;
        const bool same_count = same_device && g_mirror_nptr == nptr;
        if (!same_device) g_mirror_device = -1;  // until the uploads below have been enqueued

        // Only the parts this call uses and that differ are rewritten; nothing in the array has
        // to start at zero.  The copies are ordered before the kernel on `st`; the source is
        // pageable host memory, so each copy returns once the driver has taken the data.
        if (!same_plan) {
            desloc::fill_chunks(cfg->numel, cfg->num_tensors, chunk_elems, g_mirror.chunks, g_heads);
            std::memcpy(g_mirror_numel, cfg->numel, static_cast<size_t>(cfg->num_tensors) * sizeof(int64_t));
            std::memcpy(g_mirror_heads, g_heads, static_cast<size_t>(cfg->num_tensors) * sizeof(int64_t));
            g_mirror_nt = cfg->num_tensors;
            g_mirror_chunk_elems = chunk_elems;
            e = cudaMemcpyAsync(base + offsetof(ScratchImage, chunks), g_mirror.chunks,
                                static_cast<size_t>(nchunks) * sizeof(desloc::Chunk),
                                cudaMemcpyHostToDevice, st);
        }
        const void *const *src[4] = {reinterpret_cast<const void *const *>(x),
                                     reinterpret_cast<const void *const *>(u),
                                     reinterpret_cast<const void *const *>(v), grads};
        const size_t tbytes = static_cast<size_t>(nptr) * sizeof(void *);
        for (int arr = 0; arr < 4 && e == cudaSuccess; ++arr) {
            if (!src[arr]) continue;  // SGDM has no v table
            if (same_count && std::memcmp(g_mirror.tables[arr], src[arr], tbytes) == 0) continue;
            std::memcpy(g_mirror.tables[arr], src[arr], tbytes);
            e = cudaMemcpyAsync(base + offsetof(ScratchImage, tables) +
                                    static_cast<size_t>(arr) * kMaxPointers * sizeof(void *),
                                g_mirror.tables[arr], tbytes, cudaMemcpyHostToDevice, st);
        }
        if (e != cudaSuccess) {
            g_mirror_device = -1;  // the array's contents are no longer known
            rc = DESLOC_E_CUDA;
            break;
        }
        g_mirror_device = cuda_device;
        g_mirror_nptr = nptr;

        desloc::StepArgs a{};
        void **tab = reinterpret_cast<void **>(base + offsetof(ScratchImage, tables));
        a.chunks = reinterpret_cast<const desloc::Chunk *>(base + offsetof(ScratchImage, chunks));
        a.nchunks = nchunks;
        a.x = reinterpret_cast<float *const *>(tab);
        a.u = reinterpret_cast<float *const *>(tab + kMaxPointers);
        a.v = reinterpret_cast<float *const *>(tab + 2 * kMaxPointers);
        a.g = reinterpret_cast<const void *const *>(tab + 3 * kMaxPointers);
        a.gscale = nullptr;
        a.diag = nullptr;
        desloc::fill_hyper(a, *cfg, lr_t, clip_bound_t);
        a.direct = plan.direct ? 1 : 0;
        void *params[] = {&a};
        e = desloc::prepare_launch(plan);
        if (e == cudaSuccess)
            e = cudaLaunchKernel(plan.fn, dim3(static_cast<unsigned>(plan.grid)),
                                 dim3(desloc::BLOCK_THREADS), params, plan.smem, st);
        if (e != cudaSuccess) { rc = DESLOC_E_CUDA; break; }
    } while (false);
    if (rc == DESLOC_E_CUDA) (void)cudaGetLastError();
    if (dev_before != cuda_device) cudaSetDevice(dev_before);
    if (rc == DESLOC_OK && mask_out) *mask_out = mask;
    return rc;
}
