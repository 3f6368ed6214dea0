// moe_dispatch_noalloc: the dispatch stage for callers that cannot obtain device memory of
// their own for scratch (see include/moe.h). Its scratch is a fixed array that lives in the
// library's device image instead of a caller-provided workspace.
#include <mutex>

#include "moe_internal.cuh"

namespace {

// Fixed scratch of the chunk histograms of the counting sort. Every GPU that loads the library
// holds these 4 MiB + 256 B until the process exits. In host code this name is only a stand-in
// for the symbol, never a device address: the address is looked up once per device below.
__device__ __align__(256) int32_t g_dispatch_scratch[MOE_NOALLOC_SCRATCH_INTS];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
int32_t *g_scratch_addr[kMaxDevices];  // device address of the array, per device ordinal (nullptr: not looked up yet)

// First call on a device: look the address up, with that device current. Later calls reuse it.
int32_t scratch_for_current_device(int32_t **out) {
    int dev = -1;
    MOE_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return MOE_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_dispatch_scratch) != cudaSuccess || ptr == nullptr) return MOE_ERR_CUDA;
        g_scratch_addr[dev] = static_cast<int32_t *>(ptr);
    }
    *out = g_scratch_addr[dev];
    return MOE_OK;
}

}  // namespace

extern "C" int32_t moe_dispatch_noalloc(const moe_config *cfg, const void *x, const int32_t *topk_idx, void *xs,
                                        int32_t *perm, int32_t *inv_perm, int32_t *counts, int32_t *offsets,
                                        void *stream) {
    MOE_TRY(moe_validate(cfg));
    const void *ptrs[] = {x, topk_idx, xs, perm, inv_perm, counts, offsets};
    for (const void *p : ptrs)
        if (p == nullptr || !moe::aligned16(p)) return MOE_ERR_INVALID_ARG;
    const int64_t R = (int64_t)cfg->T * cfg->k;
    if (moe::dispatch_ws_elems(R, cfg->n) > (int64_t)MOE_NOALLOC_SCRATCH_INTS) return MOE_ERR_WORKSPACE;
    int32_t *scratch = nullptr;
    MOE_TRY(scratch_for_current_device(&scratch));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The histogram kernel writes every scratch word it later reads, so nothing has to start at zero.
    MOE_TRY(moe::launch_dispatch_index(topk_idx, R, cfg->n, perm, inv_perm, counts, offsets, scratch, st));
    return moe::launch_dispatch_rows(x, cfg->act, cfg->T, cfg->k, cfg->d, inv_perm, xs, st);
}
