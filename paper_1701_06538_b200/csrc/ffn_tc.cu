// Tensor-core expert kernels (tcgen05 / TMEM / TMA). Placeholder until the kernels land:
// reports "not supported" so the SIMT grouped GEMM is used.
#include "moe_internal.cuh"

namespace moe {
bool tc_ffn_supported(const moe_config &) { return false; }
int64_t tc_ffn_ws_bytes(const moe_config &) { return 0; }
int32_t launch_tc_ffn(const moe_config &, const void *, const int32_t *, const void *, const void *, const void *,
                      const void *, void *, void *, void *, int32_t *, cudaStream_t) {
    return MOE_ERR_UNSUPPORTED;
}
}  // namespace moe
