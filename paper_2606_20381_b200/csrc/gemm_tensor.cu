// Placeholder until the tcgen05 path is wired in: reports itself unsupported so dispatch falls back to the exact path.
#include "common.cuh"
namespace ufp4 {
size_t gemm_tensor_workspace_bytes(int64_t, int64_t, int64_t) { return 0; }
int gemm_tensor_kernel_launches() { return 0; }
bool gemm_tensor_supported(const ufp4_qtensor *, const ufp4_qtensor *, int64_t, int64_t, int64_t, int) { return false; }
int gemm_tensor_launch(const ufp4_qtensor *, const ufp4_qtensor *, void *, int64_t, int, int, int64_t, int64_t, int64_t,
                       const int64_t *, const int64_t *, int, int64_t, void *, size_t, int32_t *, void *) {
    return UFP4_ERR_UNSUPPORTED;
}
}  // namespace ufp4
