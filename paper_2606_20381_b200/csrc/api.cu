// Host-side entry points of libufp4 that are not tied to one kernel file: version, status strings, size helpers and
// the GEMM dispatch (argument validation, path selection).
#include <atomic>

#include "common.cuh"

namespace ufp4 {
// test hooks of the tensor-core launchers (ufp4_debug_wait_injection)
static std::atomic<uint32_t> g_wait_limit{0};
static std::atomic<int> g_skip_loads{0};
uint32_t debug_wait_limit() { return g_wait_limit.load(std::memory_order_relaxed); }
int debug_skip_loads() { return g_skip_loads.load(std::memory_order_relaxed); }

int gemm_exact_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int mode,
                      int64_t M, int64_t N, int64_t K, const int64_t *offsets, int num_groups, int64_t group_n,
                      void *stream);
size_t gemm_tensor_workspace_bytes(int64_t a_rows, int64_t b_rows, int64_t K);
int gemm_tensor_kernel_launches();
int gemm_noalloc_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16,
                        int32_t *dev_status, void *stream);
size_t gemm_noalloc_max_bytes();
bool gemm_tensor_supported(const ufp4_qtensor *A, const ufp4_qtensor *B, int64_t M, int64_t N, int64_t K, int mode);
struct TcQOut {
    uint8_t *row_codes, *col_codes;
    float *row_scales, *col_scales;
    int64_t row_ldc, row_lds, col_ldc, col_lds;
    int rht, pow2;
    uint32_t sign_mask;
};
int gemm_tensor_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int mode,
                       int64_t M, int64_t N, int64_t K, const int64_t *offsets, const int64_t *host_offsets,
                       int num_groups, int64_t group_n, void *workspace, size_t workspace_bytes, int32_t *dev_status,
                       void *stream, const TcQOut *qout);

size_t gemm_promote_workspace_bytes(int64_t a_rows, int64_t b_rows, int64_t K);
int gemm_promote_kernel_launches();
bool gemm_promote_supported(int mode, int64_t group_n);
int gemm_promote_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int mode,
                        int64_t M, int64_t N, int64_t K, const int64_t *offsets, int num_groups, int64_t group_n,
                        void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);

size_t gemm_split_workspace_bytes(int64_t a_rows, int64_t b_rows, int64_t K);
int gemm_split_kernel_launches();
bool gemm_split_supported(const ufp4_qtensor *A, const ufp4_qtensor *B, int64_t M, int64_t N, int64_t K, int mode);
int gemm_split_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int mode,
                      int64_t M, int64_t N, int64_t K, const int64_t *offsets, const int64_t *host_offsets, int num_groups,
                      int64_t group_n, void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream,
                      bool single);
size_t gemm_mx_workspace_bytes(int64_t a_rows, int64_t b_rows, int64_t K);
int gemm_mx_kernel_launches();
bool gemm_mx_supported(const ufp4_qtensor *A, const ufp4_qtensor *B, int64_t M, int64_t N, int64_t K, int mode);
int gemm_mx_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int mode, int64_t M,
                   int64_t N, int64_t K, const int64_t *offsets, int num_groups, int64_t group_n, void *workspace,
                   size_t workspace_bytes, int32_t *dev_status, void *stream);
size_t gemm_nvf4_workspace_bytes(const ufp4_qtensor *A, const ufp4_qtensor *B);
int gemm_nvf4_kernel_launches();
bool gemm_nvf4_supported(const ufp4_qtensor *A, const ufp4_qtensor *B, int64_t M, int64_t N, int64_t K, int mode);
int gemm_nvf4_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int64_t M, int64_t N,
                     int64_t K, void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream);
size_t gemm_fp16_workspace_bytes(int64_t a_rows, int64_t b_rows, int64_t K);
bool gemm_fp16_supported(const ufp4_qtensor *A, const ufp4_qtensor *B, int64_t M, int64_t N, int64_t K, int mode);

static int check_operand(const ufp4_qtensor *q) {
    if (!q || !q->codes || !q->scales) return UFP4_ERR_NULL;
    if (q->grid < 0 || q->grid > 4 || q->scale_fmt < 0 || q->scale_fmt > 3) return UFP4_ERR_ENUM;
    if (q->rows < 1 || q->k < 16 || q->k % 16 != 0) return UFP4_ERR_SHAPE;
    if (q->ld_codes_bytes < q->k / 2 || q->ld_codes_bytes % 16 != 0 || q->ld_scales < q->k / 16) return UFP4_ERR_ALIGN;
    if (!aligned_to(q->codes, 16)) return UFP4_ERR_ALIGN;
    if (q->scale_fmt != UFP4_SCALE_E4M3_TENSOR && !aligned_to(q->scales, 4)) return UFP4_ERR_ALIGN;
    if (q->scale_fmt == UFP4_SCALE_E4M3_TENSOR && !q->tensor_scale) return UFP4_ERR_NULL;
    return UFP4_OK;
}

static int gemm_dispatch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int path,
                         int mode, int64_t M, int64_t N, int64_t K, const int64_t *offsets, const int64_t *host_offsets,
                         int num_groups, int64_t group_n, void *workspace, size_t workspace_bytes, int32_t *dev_status,
                         void *stream) {
    if (path < 0 || path > 7) return UFP4_ERR_ENUM;
    if (!C) return UFP4_ERR_NULL;
    if (ldc < N) return UFP4_ERR_SHAPE;
    if (!aligned_to(C, 16) || (ldc * (c_is_bf16 ? 2 : 4)) % 16 != 0) return UFP4_ERR_ALIGN;
    const bool tensor_ok = gemm_tensor_supported(A, B, M, N, K, mode);
    if (path == UFP4_PATH_TENSOR && !tensor_ok) return UFP4_ERR_UNSUPPORTED;
    if (path == UFP4_PATH_EXACT)
        return gemm_exact_launch(A, B, C, ldc, c_is_bf16, mode, M, N, K, offsets, num_groups, group_n, stream);
    // MX (hardware block scaling): on request only; the folded path is the faster one on the same operands
    if (path == UFP4_PATH_MX) {
        if (!gemm_mx_supported(A, B, M, N, K, mode)) return UFP4_ERR_UNSUPPORTED;
        if (!workspace || workspace_bytes < gemm_mx_workspace_bytes(A->rows, B->rows, A->k)) return UFP4_ERR_WORKSPACE;
        return gemm_mx_launch(A, B, C, ldc, c_is_bf16, mode, M, N, K, offsets, num_groups, group_n, workspace,
                              workspace_bytes, dev_status, stream);
    }
    if (path == UFP4_PATH_TENSOR || (path == UFP4_PATH_AUTO && tensor_ok)) {
        const size_t need = gemm_tensor_workspace_bytes(A->rows, B->rows, A->k);
        if (workspace && workspace_bytes >= need)
            return gemm_tensor_launch(A, B, C, ldc, c_is_bf16, mode, M, N, K, offsets, host_offsets, num_groups, group_n,
                                      workspace, workspace_bytes, dev_status, stream, nullptr);
        if (path == UFP4_PATH_TENSOR) return UFP4_ERR_WORKSPACE;
    }
    // NVF4 (native FP4 with hardware UE4M3 scales): E4M3 x tensor scales on both operands, plain products; what AUTO takes
    // for those (measured faster than FP16 with one, two or four MMAs per step)
    const bool nvf4_ok = gemm_nvf4_supported(A, B, M, N, K, mode);
    const bool nvf4_auto = nvf4_ok;
    if (path == UFP4_PATH_NVF4 && !nvf4_ok) return UFP4_ERR_UNSUPPORTED;
    if (path == UFP4_PATH_NVF4 || (path == UFP4_PATH_AUTO && nvf4_auto)) {
        if (workspace && workspace_bytes >= gemm_nvf4_workspace_bytes(A, B))
            return gemm_nvf4_launch(A, B, C, ldc, c_is_bf16, M, N, K, workspace, workspace_bytes, dev_status, stream);
        if (path == UFP4_PATH_NVF4) return UFP4_ERR_WORKSPACE;
    }
    // FP16 (one piece): E4M3 x tensor scales on both operands
    const bool fp16_ok = gemm_fp16_supported(A, B, M, N, K, mode);
    if (path == UFP4_PATH_FP16 && !fp16_ok) return UFP4_ERR_UNSUPPORTED;
    if (path == UFP4_PATH_FP16 || (path == UFP4_PATH_AUTO && fp16_ok)) {
        const size_t need = gemm_fp16_workspace_bytes(A->rows, B->rows, A->k);
        if (workspace && workspace_bytes >= need)
            return gemm_split_launch(A, B, C, ldc, c_is_bf16, mode, M, N, K, offsets, host_offsets, num_groups, group_n,
                                     workspace, workspace_bytes, dev_status, stream, true);
        if (path == UFP4_PATH_FP16) return UFP4_ERR_WORKSPACE;
    }
    // SPLIT, or AUTO for scale formats the folded path cannot take
    const bool split_ok = gemm_split_supported(A, B, M, N, K, mode);
    if (path == UFP4_PATH_SPLIT && !split_ok) return UFP4_ERR_UNSUPPORTED;
    if (path == UFP4_PATH_SPLIT || (path == UFP4_PATH_AUTO && split_ok)) {
        const size_t need = gemm_split_workspace_bytes(A->rows, B->rows, A->k);
        if (workspace && workspace_bytes >= need)
            return gemm_split_launch(A, B, C, ldc, c_is_bf16, mode, M, N, K, offsets, host_offsets, num_groups, group_n,
                                     workspace, workspace_bytes, dev_status, stream, false);
        if (path == UFP4_PATH_SPLIT) return UFP4_ERR_WORKSPACE;
    }
    // PROMOTE, or AUTO for what neither tensor-core operand form can take
    const bool promote_ok = gemm_promote_supported(mode, group_n);
    if (path == UFP4_PATH_PROMOTE && !promote_ok) return UFP4_ERR_UNSUPPORTED;
    if (promote_ok) {
        const size_t need = gemm_promote_workspace_bytes(A->rows, B->rows, A->k);
        if (workspace && workspace_bytes >= need)
            return gemm_promote_launch(A, B, C, ldc, c_is_bf16, mode, M, N, K, offsets, num_groups, group_n, workspace,
                                       workspace_bytes, dev_status, stream);
        if (path == UFP4_PATH_PROMOTE) return UFP4_ERR_WORKSPACE;
    }
    return gemm_exact_launch(A, B, C, ldc, c_is_bf16, mode, M, N, K, offsets, num_groups, group_n, stream);
}

}  // namespace ufp4

extern "C" int ufp4_version(void) { return 200; }

extern "C" const char *ufp4_status_string(int status) {
    switch (status) {
        case UFP4_OK: return "ok";
        case UFP4_ERR_NULL: return "a required pointer is NULL";
        case UFP4_ERR_SHAPE: return "bad shape: a dimension is non-positive or not a multiple of what the operation needs";
        case UFP4_ERR_ALIGN: return "bad alignment of a pointer or leading dimension";
        case UFP4_ERR_ENUM: return "enum value out of range";
        case UFP4_ERR_UNSUPPORTED: return "combination not supported by this build";
        case UFP4_ERR_CUDA: return "a CUDA runtime call failed";
        case UFP4_ERR_WORKSPACE: return "workspace missing or too small";
        default: return "unknown status";
    }
}

extern "C" int ufp4_qtensor_bytes(int64_t rows, int64_t k, int scale_fmt, size_t *codes_bytes, size_t *scales_bytes) {
    if (!codes_bytes || !scales_bytes) return UFP4_ERR_NULL;
    if (rows < 1 || k < 16 || k % 16 != 0) return UFP4_ERR_SHAPE;
    if (scale_fmt < 0 || scale_fmt > 3) return UFP4_ERR_ENUM;
    int64_t ld = (k / 2 + 15) / 16 * 16;
    *codes_bytes = (size_t)(rows * ld);
    *scales_bytes = (size_t)(rows * (k / 16) * (scale_fmt == UFP4_SCALE_E4M3_TENSOR ? 1 : 4));
    return UFP4_OK;
}

extern "C" size_t ufp4_gemm_workspace_bytes(const ufp4_qtensor *A, const ufp4_qtensor *B, int path) {
    if (!A || !B || path == UFP4_PATH_EXACT) return 0;
    const bool pow2 = ufp4::is_pow2_fmt(A->scale_fmt) && ufp4::is_pow2_fmt(B->scale_fmt);
    if (path == UFP4_PATH_MX) return pow2 ? ufp4::gemm_mx_workspace_bytes(A->rows, B->rows, A->k) : 0;
    if (path == UFP4_PATH_TENSOR || (path == UFP4_PATH_AUTO && pow2))
        return pow2 ? ufp4::gemm_tensor_workspace_bytes(A->rows, B->rows, A->k) : 0;
    const bool e4m3 = A->scale_fmt == UFP4_SCALE_E4M3_TENSOR && B->scale_fmt == UFP4_SCALE_E4M3_TENSOR;
    if (path == UFP4_PATH_NVF4) return e4m3 ? ufp4::gemm_nvf4_workspace_bytes(A, B) : 0;
    if (path == UFP4_PATH_FP16) return e4m3 ? ufp4::gemm_fp16_workspace_bytes(A->rows, B->rows, A->k) : 0;
    // AUTO takes FP16 for E4M3 x tensor scales, else SPLIT, and PROMOTE only where SPLIT does not apply: the two-piece
    // workspace is enough for all of them
    const size_t split = ufp4::gemm_split_workspace_bytes(A->rows, B->rows, A->k);
    const size_t promote = ufp4::gemm_promote_workspace_bytes(A->rows, B->rows, A->k);
    if (path == UFP4_PATH_SPLIT) return split;
    if (path == UFP4_PATH_PROMOTE) return promote;
    const size_t nvf4 = e4m3 ? ufp4::gemm_nvf4_workspace_bytes(A, B) : 0;      // what AUTO takes for plain products
    const size_t m = split > promote ? split : promote;
    return m > nvf4 ? m : nvf4;
}

extern "C" int ufp4_gemm_path_taken(const ufp4_qtensor *A, const ufp4_qtensor *B, int path, int *kernel_launches) {
    int rc = ufp4::check_operand(A);
    if (rc != UFP4_OK) return rc;
    rc = ufp4::check_operand(B);
    if (rc != UFP4_OK) return rc;
    if (path < 0 || path > 7) return UFP4_ERR_ENUM;
    if (A->k != B->k) return UFP4_ERR_SHAPE;
    if (path == UFP4_PATH_MX && !ufp4::gemm_mx_supported(A, B, A->rows, B->rows, A->k, 0)) return UFP4_ERR_UNSUPPORTED;
    bool tensor_ok = ufp4::gemm_tensor_supported(A, B, A->rows, B->rows, A->k, 0);
    bool split_ok = ufp4::gemm_split_supported(A, B, A->rows, B->rows, A->k, 0);
    bool fp16_ok = ufp4::gemm_fp16_supported(A, B, A->rows, B->rows, A->k, 0);
    bool nvf4_ok = ufp4::gemm_nvf4_supported(A, B, A->rows, B->rows, A->k, 0);
    bool nvf4_auto = nvf4_ok;
    if (path == UFP4_PATH_NVF4 && !nvf4_ok) return UFP4_ERR_UNSUPPORTED;
    if (path == UFP4_PATH_TENSOR && !tensor_ok) return UFP4_ERR_UNSUPPORTED;
    if (path == UFP4_PATH_SPLIT && !split_ok) return UFP4_ERR_UNSUPPORTED;
    if (path == UFP4_PATH_FP16 && !fp16_ok) return UFP4_ERR_UNSUPPORTED;
    int taken = path == UFP4_PATH_EXACT ? UFP4_PATH_EXACT
              : path == UFP4_PATH_MX ? UFP4_PATH_MX
              : (path == UFP4_PATH_TENSOR || (path == UFP4_PATH_AUTO && tensor_ok)) ? UFP4_PATH_TENSOR
              : (path == UFP4_PATH_NVF4 || (path == UFP4_PATH_AUTO && nvf4_auto)) ? UFP4_PATH_NVF4
              : (path == UFP4_PATH_FP16 || (path == UFP4_PATH_AUTO && fp16_ok)) ? UFP4_PATH_FP16
              : (path == UFP4_PATH_SPLIT || (path == UFP4_PATH_AUTO && split_ok)) ? UFP4_PATH_SPLIT : UFP4_PATH_PROMOTE;
    if (kernel_launches)
        *kernel_launches = taken == UFP4_PATH_EXACT ? 1 : taken == UFP4_PATH_MX ? ufp4::gemm_mx_kernel_launches()
                         : taken == UFP4_PATH_NVF4 ? ufp4::gemm_nvf4_kernel_launches()
                         : taken == UFP4_PATH_TENSOR ? ufp4::gemm_tensor_kernel_launches()
                         : (taken == UFP4_PATH_SPLIT || taken == UFP4_PATH_FP16) ? ufp4::gemm_split_kernel_launches()
                                                    : ufp4::gemm_promote_kernel_launches();
    return taken;
}

extern "C" int ufp4_gemm(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int layout,
                         int path, void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream) {
    int rc = ufp4::check_operand(A);
    if (rc != UFP4_OK) return rc;
    rc = ufp4::check_operand(B);
    if (rc != UFP4_OK) return rc;
    if (layout < 0 || layout > 2) return UFP4_ERR_ENUM;
    if (A->k != B->k) return UFP4_ERR_SHAPE;
    return ufp4::gemm_dispatch(A, B, C, ldc, c_is_bf16, path, 0, A->rows, B->rows, A->k, nullptr, nullptr, 1, B->rows,
                               workspace, workspace_bytes, dev_status, stream);
}

extern "C" int ufp4_gemm_grouped(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16,
                                 int layout, int path, const int64_t *offsets, const int64_t *host_offsets,
                                 int num_groups, int64_t group_n, void *workspace, size_t workspace_bytes,
                                 int32_t *dev_status, void *stream) {
    int rc = ufp4::check_operand(A);
    if (rc != UFP4_OK) return rc;
    rc = ufp4::check_operand(B);
    if (rc != UFP4_OK) return rc;
    if (layout < 0 || layout > 2) return UFP4_ERR_ENUM;
    if (!offsets || !host_offsets) return UFP4_ERR_NULL;
    if (num_groups < 1 || A->k != B->k) return UFP4_ERR_SHAPE;
    if (host_offsets[0] != 0) return UFP4_ERR_SHAPE;
    for (int g = 0; g < num_groups; ++g)
        if (host_offsets[g + 1] < host_offsets[g] || host_offsets[g + 1] % 128 != 0) return UFP4_ERR_SHAPE;
    const int64_t total = host_offsets[num_groups];
    if (layout == UFP4_BWD_DW) {
        // reduction grouped: A [N][total], B [Kout][total], C [num_groups * N][Kout]
        if (A->k != total) return UFP4_ERR_SHAPE;
        return ufp4::gemm_dispatch(A, B, C, ldc, c_is_bf16, path, 2, A->rows, B->rows, A->k, offsets, host_offsets,
                                   num_groups, group_n, workspace, workspace_bytes, dev_status, stream);
    }
    // rows grouped: A [total][K], B [num_groups * group_n][K], C [total][group_n]
    if (A->rows != total || group_n < 1 || B->rows != (int64_t)num_groups * group_n) return UFP4_ERR_SHAPE;
    return ufp4::gemm_dispatch(A, B, C, ldc, c_is_bf16, path, 1, A->rows, group_n, A->k, offsets, host_offsets,
                               num_groups, group_n, workspace, workspace_bytes, dev_status, stream);
}

extern "C" size_t ufp4_gemm_noalloc_max_scratch_bytes(void) { return ufp4::gemm_noalloc_max_bytes(); }

extern "C" int ufp4_gemm_noalloc(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16,
                                 int32_t *dev_status, void *stream) {
    int rc = ufp4::check_operand(A);
    if (rc != UFP4_OK) return rc;
    rc = ufp4::check_operand(B);
    if (rc != UFP4_OK) return rc;
    if (!C) return UFP4_ERR_NULL;
    if (A->k != B->k || ldc < B->rows) return UFP4_ERR_SHAPE;
    if (!ufp4::aligned_to(C, 16) || (ldc * (c_is_bf16 ? 2 : 4)) % 16 != 0) return UFP4_ERR_ALIGN;
    return ufp4::gemm_noalloc_launch(A, B, C, ldc, c_is_bf16, dev_status, stream);
}

extern "C" int ufp4_debug_wait_injection(uint32_t poll_limit, int skip_loads) {
    if (skip_loads != 0 && skip_loads != 1) return UFP4_ERR_ENUM;
    ufp4::g_wait_limit.store(poll_limit, std::memory_order_relaxed);
    ufp4::g_skip_loads.store(skip_loads, std::memory_order_relaxed);
    return UFP4_OK;
}

extern "C" int ufp4_gemm_quantized(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C_bf16, int64_t ldc, int rht_block,
                                   uint64_t seed_rht, const ufp4_qtensor *out_row, const ufp4_qtensor *out_col,
                                   void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream) {
    int rc = ufp4::check_operand(A);
    if (rc != UFP4_OK) return rc;
    rc = ufp4::check_operand(B);
    if (rc != UFP4_OK) return rc;
    if (A->k != B->k) return UFP4_ERR_SHAPE;
    if (rht_block != 0 && rht_block != 16) return UFP4_ERR_UNSUPPORTED;
    if (!out_row && !out_col) return UFP4_ERR_NULL;
    const int64_t M = A->rows, N = B->rows;
    if (M % 16 != 0 || N % 16 != 0) return UFP4_ERR_SHAPE;
    if (!ufp4::gemm_tensor_supported(A, B, M, N, A->k, 0)) return UFP4_ERR_UNSUPPORTED;
    const ufp4_qtensor *any = out_row ? out_row : out_col;
    const int fmt = any->scale_fmt;
    if (fmt != UFP4_SCALE_FP32 && fmt != UFP4_SCALE_POW2) return UFP4_ERR_UNSUPPORTED;
    for (int v = 0; v < 2; ++v) {
        const ufp4_qtensor *q = v ? out_col : out_row;
        if (!q) continue;
        if (!q->codes || !q->scales) return UFP4_ERR_NULL;
        if (q->grid != UFP4_GRID_INT4 || q->scale_fmt != fmt) return UFP4_ERR_UNSUPPORTED;
        if (q->rows != (v ? N : M) || q->k != (v ? M : N)) return UFP4_ERR_SHAPE;
        if (q->ld_codes_bytes < q->k / 2 || q->ld_codes_bytes % 16 != 0 || q->ld_scales < q->k / 16 ||
            !ufp4::aligned_to(q->codes, 16) || !ufp4::aligned_to(q->scales, 4))
            return UFP4_ERR_ALIGN;
    }
    if (C_bf16) {
        if (ldc < N) return UFP4_ERR_SHAPE;
        if (!ufp4::aligned_to(C_bf16, 16) || (ldc * 2) % 16 != 0) return UFP4_ERR_ALIGN;
    }
    if (!workspace || workspace_bytes < ufp4::gemm_tensor_workspace_bytes(A->rows, B->rows, A->k)) return UFP4_ERR_WORKSPACE;
    ufp4::TcQOut q = {};
    if (out_row) {
        q.row_codes = static_cast<uint8_t *>(out_row->codes); q.row_scales = static_cast<float *>(out_row->scales);
        q.row_ldc = out_row->ld_codes_bytes; q.row_lds = out_row->ld_scales;
    }
    if (out_col) {
        q.col_codes = static_cast<uint8_t *>(out_col->codes); q.col_scales = static_cast<float *>(out_col->scales);
        q.col_ldc = out_col->ld_codes_bytes; q.col_lds = out_col->ld_scales;
    }
    q.rht = rht_block == 16;
    q.pow2 = fmt == UFP4_SCALE_POW2;
    q.sign_mask = ufp4_rht_sign_mask(seed_rht);
    return ufp4::gemm_tensor_launch(A, B, C_bf16, C_bf16 ? ldc : N, 1, 0, M, N, A->k, nullptr, nullptr, 1, N, workspace,
                                    workspace_bytes, dev_status, stream, &q);
}
