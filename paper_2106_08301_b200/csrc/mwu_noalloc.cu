// mwu_project_static: the projection for callers that must not allocate device memory.
//
// Some hosts of this library may not call cudaMalloc at the point where they need a projection:
// a plug-in running inside an engine that owns the whole memory pool, a training loop whose
// memory budget is frozen after start-up (an allocation there can fail or stall every stream of
// the device while the driver maps memory), or code that simply has no allocator handle to ask.
// mwu_project needs a scratch buffer from its caller; this variant brings its own: a fixed array
// that lives in the library's device image, so every GPU that loads the library holds it until
// the process exits.  Nothing in here calls cudaMalloc, cudaFree or any allocating routine.
#include <mutex>

#include "mwu_common.cuh"

namespace {

// Enough for MWU_STATIC_MAX_BLOCKS blocks: 4 bytes of bin codes per block, 8 bytes per entry of
// the candidate list (a quarter of the blocks) and the fixed selection state (histograms, sort
// buffers) of mwu_project, which is under 1.5 MiB.
constexpr size_t kScratchBytes = (size_t)1536 * 1024 + 4 * ((size_t)MWU_STATIC_MAX_BLOCKS + 8) +
                                 8 * ((size_t)MWU_STATIC_MAX_BLOCKS / 4 + 4096) + 1024;

static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

// In host code `g_scratch` is only a handle for the runtime, not an address a kernel can use;
// the device address is looked up once per device and remembered here.
constexpr int kMaxDevices = 64;
void *g_scratch_addr[kMaxDevices] = {};
std::mutex g_setup_lock;

int scratch_for_current_device(void **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return MWU_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return MWU_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> guard(g_setup_lock);
    if (!g_scratch_addr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_scratch) != cudaSuccess || !ptr) return MWU_ERR_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return MWU_OK;
}

}  // namespace

extern "C" int mwu_project_static(const mwu_proj_desc *desc, const float *W, const float *U_dual,
                                  float *Q, float *u, uint32_t *pruned_bitmap,
                                  uint32_t *unified_bitmap, uint32_t *sign_bits, double *loss_u,
                                  double *loss_p, uint32_t *dev_status, void *cuda_stream) {
    const int rc = mwu::validate_desc(desc, false);
    if (rc != MWU_OK) return rc;
    const int64_t n_blocks = mwu::shape_of(desc).mb;
    const size_t need = mwu_project_workspace_bytes(desc);
    if (n_blocks > (int64_t)MWU_STATIC_MAX_BLOCKS || need == 0 || need > kScratchBytes)
        return MWU_ERR_WORKSPACE;            // tensor too large for the built-in scratch
    void *scratch = nullptr;
    const int src = scratch_for_current_device(&scratch);
    if (src != MWU_OK) return src;
    // mwu_project zeroes the part of the scratch that has to start at zero (selection state and
    // histograms) on the caller's stream before its first kernel, so what the previous call left
    // behind does not matter.
    return mwu_project(desc, W, U_dual, Q, u, pruned_bitmap, unified_bitmap, sign_bits, loss_u,
                       loss_p, dev_status, scratch, kScratchBytes, cuda_stream);
}
