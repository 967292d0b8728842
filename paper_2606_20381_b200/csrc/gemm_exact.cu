// Exact block-scaled 4-bit GEMM (Sec. 2.2: Y^ = Q_G(XH') Q_G(WH')^T on dequantized values).
//
// C[m][n] = sum_kb sA[m][kb] * sB[n][kb] * P_kb[m][n],  P_kb = sum over the 16 codes of block kb of qa * qb (integer).
// The integer partial of every 16-block is formed exactly with 8-bit dot products and promoted with the product of the
// two FP32 block scales, so this path is valid for every grid and scale format.  Four promoted blocks are summed in
// FP32 and the running sum is kept in FP64, which keeps the error independent of K (a few 2^-24 of sum |a_k b_k|).
// The per-16 promotion runs on the CUDA cores: this path is bounded by FP32 issue rate, not by the tensor cores.
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "common.cuh"

namespace ufp4 {

constexpr int kBM = 64, kBN = 64, kBK = 64;   // CTA tile; kBK = 4 quant blocks
constexpr int kPitch = kBK + 16;               // bytes per decoded row in shared memory (+16 against bank conflicts)

struct OperandView {
    const uint8_t *codes;
    const void *scales;
    const float *tensor_scale;
    int64_t ldc, lds;
    int grid, sfmt;
};

struct ExactParams {
    OperandView A, B;
    void *C;
    int64_t ldc;
    int c_is_bf16;
    int64_t M, N, K;       // per-group problem: C tile space is M x N, reduction K (whole K unless K-grouped)
    int mode;              // 0 plain, 1 rows of A grouped (fwd_y / bwd_dx), 2 reduction grouped (bwd_dw)
    const int64_t *offsets;
    int num_groups;
    int64_t group_n;
};

// Signed 8-bit value of a nibble in units of `unit`: INT4 q (unit 1), E1M2 q (unit 1/4), E2M1 2*value (unit 1/2).
__device__ __forceinline__ int decode_nibble(int grid, uint32_t nib) {
    if (grid == UFP4_GRID_INT4) return (int)(nib ^ 8u) - 8;
    int mag;
    if (grid == UFP4_GRID_E1M2) mag = nib & 7;
    else {
        const int idx = nib & 7;   // 2 * {0, .5, 1, 1.5, 2, 3, 4, 6} = {0, 1, 2, 3, 4, 6, 8, 12}
        mag = idx < 2 ? idx : (2 + (idx & 1)) << ((idx >> 1) - 1);
    }
    return (nib & 8u) ? -mag : mag;
}

__device__ __forceinline__ float unit_of(int grid) {
    return grid == UFP4_GRID_INT4 ? 1.0f : (grid == UFP4_GRID_E1M2 ? 0.25f : 0.5f);
}

__device__ __forceinline__ float load_scale(const OperandView &V, int64_t row, int64_t kb, float ts) {
    if (V.sfmt == UFP4_SCALE_E4M3_TENSOR) {
        uint8_t byte = static_cast<const uint8_t *>(V.scales)[row * V.lds + kb];
        __half_raw hr = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)byte, __NV_E4M3);
        return __fmul_rn(ts, __half2float(*reinterpret_cast<__half *>(&hr)));
    }
    return static_cast<const float *>(V.scales)[row * V.lds + kb];
}

// Decode rows [r0, r0+64) x k-range [k0, k0+64) of an operand into shared memory (int8) plus its 4 scales per row.
__device__ __forceinline__ void stage_operand(const OperandView &V, int64_t r0, int64_t rmax, int64_t k0, int64_t kend,
                                              float ts, int8_t (*dst)[kPitch], float (*sdst)[4], int tid) {
    // 64 rows x 8 words of 8 codes: 512 items over 256 threads
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        int item = it * 256 + tid, r = item >> 3, wq = item & 7;
        int64_t gr = r0 + r, gk = k0 + 8 * wq;
        uint32_t w = 0;
        if (gr < rmax && gk < kend) w = *reinterpret_cast<const uint32_t *>(V.codes + gr * V.ldc + (gk >> 1));
        uint32_t lo = 0, hi = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            lo |= ((uint32_t)decode_nibble(V.grid, (w >> (4 * j)) & 0xFu) & 0xFFu) << (8 * j);
            hi |= ((uint32_t)decode_nibble(V.grid, (w >> (4 * j + 16)) & 0xFu) & 0xFFu) << (8 * j);
        }
        *reinterpret_cast<uint2 *>(&dst[r][8 * wq]) = make_uint2(lo, hi);
    }
    {
        int r = tid >> 2, kb = tid & 3;
        int64_t gr = r0 + r, gk = k0 + 16 * kb;
        float s = 0.0f;
        if (gr < rmax && gk < kend) s = load_scale(V, gr, gk >> 4, ts) * unit_of(V.grid);
        sdst[r][kb] = s;
    }
}

__global__ void __launch_bounds__(256) gemm_exact_kernel(const ExactParams P) {
    __shared__ __align__(16) int8_t As[kBM][kPitch];
    __shared__ __align__(16) int8_t Bs[kBN][kPitch];
    __shared__ float sAs[kBM][4], sBs[kBN][4];

    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int64_t m0 = (int64_t)blockIdx.y * kBM, n0 = (int64_t)blockIdx.x * kBN;
    int64_t kbeg = 0, kend = P.K, b_row_base = 0, c_row_base = 0;
    if (P.mode == 1) {
        // find the group of this row tile (offsets are multiples of 128, so a 64-row tile never straddles groups)
        int lo = 0, hi = P.num_groups;
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (P.offsets[mid] <= m0) lo = mid; else hi = mid;
        }
        b_row_base = (int64_t)lo * P.group_n;
    } else if (P.mode == 2) {
        const int g = blockIdx.z;
        kbeg = P.offsets[g];
        kend = P.offsets[g + 1];
        c_row_base = (int64_t)g * P.M;
    }
    const float tsA = P.A.sfmt == UFP4_SCALE_E4M3_TENSOR ? *P.A.tensor_scale : 1.0f;
    const float tsB = P.B.sfmt == UFP4_SCALE_E4M3_TENSOR ? *P.B.tensor_scale : 1.0f;

    double acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;

    for (int64_t k0 = kbeg; k0 < kend; k0 += kBK) {
        __syncthreads();
        stage_operand(P.A, m0, P.M, k0, kend, tsA, As, sAs, tid);
        stage_operand(P.B, b_row_base + n0, b_row_base + P.N, k0, kend, tsB, Bs, sBs, tid);
        __syncthreads();
        float c32[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) c32[i][j] = 0.0f;
#pragma unroll
        for (int kb = 0; kb < 4; ++kb) {
            int4 a[4], b[4];
            float sa[4], sb[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                a[i] = *reinterpret_cast<const int4 *>(&As[ty * 4 + i][16 * kb]);
                sa[i] = sAs[ty * 4 + i][kb];
                b[i] = *reinterpret_cast<const int4 *>(&Bs[tx * 4 + i][16 * kb]);
                sb[i] = sBs[tx * 4 + i][kb];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    int p = __dp4a(a[i].x, b[j].x, 0);
                    p = __dp4a(a[i].y, b[j].y, p);
                    p = __dp4a(a[i].z, b[j].z, p);
                    p = __dp4a(a[i].w, b[j].w, p);
                    c32[i][j] = __fmaf_rn(__int2float_rn(p), __fmul_rn(sa[i], sb[j]), c32[i][j]);
                }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] += (double)c32[i][j];
    }

#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int64_t m = m0 + ty * 4 + i;
        if (m >= P.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int64_t n = n0 + tx * 4 + j;
            if (n >= P.N) continue;
            float val = (float)acc[i][j];
            if (P.c_is_bf16) static_cast<__nv_bfloat16 *>(P.C)[(c_row_base + m) * P.ldc + n] = __float2bfloat16_rn(val);
            else static_cast<float *>(P.C)[(c_row_base + m) * P.ldc + n] = val;
        }
    }
}

int gemm_exact_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int mode,
                      int64_t M, int64_t N, int64_t K, const int64_t *offsets, int num_groups, int64_t group_n,
                      void *stream) {
    ExactParams P = {};
    P.A = OperandView{static_cast<const uint8_t *>(A->codes), A->scales, A->tensor_scale, A->ld_codes_bytes, A->ld_scales,
                      codebook_of(A->grid), A->scale_fmt};
    P.B = OperandView{static_cast<const uint8_t *>(B->codes), B->scales, B->tensor_scale, B->ld_codes_bytes, B->ld_scales,
                      codebook_of(B->grid), B->scale_fmt};
    P.C = C; P.ldc = ldc; P.c_is_bf16 = c_is_bf16;
    P.M = M; P.N = N; P.K = K; P.mode = mode;
    P.offsets = offsets; P.num_groups = num_groups; P.group_n = group_n;
    const int64_t gx = (N + kBN - 1) / kBN, gy = (M + kBM - 1) / kBM, gz = (mode == 2) ? num_groups : 1;
    if (gy > 65535 || gz > 65535 || gx > 0x7FFFFFFF || gx < 1 || gy < 1 || gz < 1) return UFP4_ERR_SHAPE;
    gemm_exact_kernel<<<dim3((unsigned)gx, (unsigned)gy, (unsigned)gz), 256, 0, static_cast<cudaStream_t>(stream)>>>(P);
    return cudaGetLastError() == cudaSuccess ? UFP4_OK : UFP4_ERR_CUDA;
}

}  // namespace ufp4
