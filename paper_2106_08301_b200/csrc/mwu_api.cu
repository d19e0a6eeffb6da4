// Small host-side entry points and the device check shared by all calls.
#include <atomic>

#include "mwu_common.cuh"

namespace mwu {

static std::atomic<unsigned long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

int check_device(int *sm_count) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return MWU_ERR_CUDA;
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return MWU_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return MWU_ERR_CUDA;
    if (major != 10) return MWU_ERR_UNSUPPORTED_DEVICE;
    if (sm_count) *sm_count = sms;
    return MWU_OK;
}

}  // namespace mwu

extern "C" const char *mwu_status_string(int status) {
    switch (status) {
        case MWU_OK: return "ok";
        case MWU_ERR_INVALID_ARG: return "invalid argument";
        case MWU_ERR_SHAPE: return "unsupported shape, block width or block counts";
        case MWU_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
        case MWU_ERR_WORKSPACE: return "workspace or output buffer too small";
        case MWU_ERR_UNSUPPORTED_DEVICE: return "device is not compute capability 10.x";
        case MWU_ERR_CUDA: return "CUDA call failed";
        default: return "unknown status";
    }
}

extern "C" uint64_t mwu_kernel_launches(void) {
    return (uint64_t)mwu::g_launches.load(std::memory_order_relaxed);
}

extern "C" int64_t mwu_count_from_permille(int64_t n_blocks, int32_t permille) {
    if (n_blocks < 0 || permille < 0) return -1;
    return (int64_t)(((__int128)permille * (__int128)n_blocks + 500) / 1000);
}
