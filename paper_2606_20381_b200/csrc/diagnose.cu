// Tensor diagnostics of a quantized tensor (not on the training hot path; used by the quantizer sweep): the operand
// projection alpha of Sec. 3.2 (Eq. 3), the normalised MSE and the level counts behind the effective bucket ratio of
// Sec. 3.3 (Eq. 6, Eq. 7), and the per-level mean signed rounding error of Sec. 3.1 (the Shrinkage-Bias measurement).
//
// One pass over the BF16 matrix and its row variant: every thread walks 16-element blocks, recomputes x' = x H'_16 with
// the quantizer's FP32 butterflies, and accumulates 19 sums; CTA partials go to the caller's workspace and a second,
// single-CTA kernel adds them in a fixed order, so the result does not depend on scheduling.
#include <math.h>

#include "common.cuh"

namespace ufp4 {

constexpr int kDiagThreads = 256;
constexpr int kDiagSums = 19;      // sum x'^2, sum (xq - x')^2, sum xq x', count[8], sum of (level - t) per level [8]

struct DiagParams {
    const uint16_t *x;
    int64_t rows, cols, ld;
    const uint8_t *codes;
    const float *scales;
    int64_t ldc, lds;
    int grid, rht;
    int load256;                   // x and its row pitch are 32-byte aligned: 256-bit loads
    uint32_t signs[4];             // bit i of the 128: eps_i = -1 (the first 16 bits serve the 16-point transform)
    int xb;                        // log2(rht_block / 16): butterfly stages that pair 16-element blocks
    float norm;                    // 1/4, or RN(1 / sqrt(rht_block)) for the wider blocks
    double *partials;              // [gridDim.x][kDiagSums]
};

__device__ __forceinline__ void diag_butterflies(float (&v)[16]) {
#pragma unroll
    for (int h = 1; h < 16; h <<= 1) {
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            if ((i & h) == 0) {
                const float a = v[i], b = v[i + h];
                v[i] = __fadd_rn(a, b);
                v[i + h] = __fsub_rn(a, b);
            }
        }
    }
}

template <int GRID>
__global__ void __launch_bounds__(kDiagThreads) diagnose_kernel(const DiagParams P) {
    __shared__ double red[kDiagThreads / 32][kDiagSums];
    __shared__ float lvl[8][kDiagThreads];         // per thread and level: sum of (level - t); column = thread, no conflicts
    const int64_t nblk = P.rows * (P.cols >> 4), bpr = P.cols >> 4;
    double sxx = 0.0, see = 0.0, sxq = 0.0;
    int cnt[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { cnt[k] = 0; lvl[k][threadIdx.x] = 0.0f; }

    // warp-uniform trip count: with an RHT block wider than 16 the eight (or fewer) neighbouring lanes that hold one
    // block's 16-element pieces exchange registers, so every lane of a warp runs every iteration (a lane past the end
    // works on zeros and adds nothing); rows hold whole RHT blocks, so a group of lanes never straddles two rows
    const int lane0 = threadIdx.x & ~31;
    for (int64_t base = (int64_t)blockIdx.x * kDiagThreads + lane0; base < nblk; base += (int64_t)gridDim.x * kDiagThreads) {
        const int64_t blk_raw = base + (threadIdx.x & 31);
        const bool valid = blk_raw < nblk;
        const int64_t blk = valid ? blk_raw : 0;
        const int64_t r = blk / bpr, b = blk - r * bpr;
        const uint4 *src = reinterpret_cast<const uint4 *>(P.x + r * P.ld + 16 * b);
        uint4 d0, d1;
        if (P.load256) {
            asm volatile("ld.global.nc.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                         : "=r"(d0.x), "=r"(d0.y), "=r"(d0.z), "=r"(d0.w), "=r"(d1.x), "=r"(d1.y), "=r"(d1.z), "=r"(d1.w) : "l"(src));
        } else {
            d0 = __ldg(src);
            d1 = __ldg(src + 1);
        }
        const uint2 cw = __ldg(reinterpret_cast<const uint2 *>(P.codes + r * P.ldc + 8 * b));
        const float s = valid ? __ldg(P.scales + r * P.lds + b) : 0.0f;
        const uint32_t w[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
        float v[16];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            v[2 * j] = __uint_as_float(w[j] << 16);
            v[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
        }
        if (P.rht) {
            const int j = (int)b & ((1 << P.xb) - 1);              // this block's place inside its RHT block
            const uint32_t sb = P.signs[j >> 1] >> (16 * (j & 1));
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(__float_as_uint(v[i]) ^ (((sb >> i) & 1u) << 31));
            diag_butterflies(v);
            for (int st = 0; st < P.xb; ++st) {
                const int m = 1 << st;
                const bool upper = (j & m) != 0;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float o = __shfl_xor_sync(0xFFFFFFFFu, v[i], m);
                    v[i] = upper ? __fsub_rn(o, v[i]) : __fadd_rn(v[i], o);
                }
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = __fmul_rn(v[i], P.norm);
        }
        if (!valid) continue;                                      // uniform exchanges are done: nothing to add
        const float inv_s = s > 0.0f ? 1.0f / s : 0.0f;          // t only feeds an average: a rounded reciprocal is fine
        uint64_t hist = 0;                                      // one byte per level: this block's counts
        float bxx = 0.0f, bee = 0.0f, bxq = 0.0f;               // the block's three sums in FP32 (16 terms), FP64 across blocks
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t nib = ((i < 8 ? cw.x : cw.y) >> (4 * (i & 7))) & 0xFu;
            // magnitude level index and signed value in grid units
            int idx;
            float val;
            if (GRID == UFP4_GRID_INT4) {
                const int q = (int)(nib ^ 8u) - 8;
                idx = q == -8 ? 0 : abs(q);          // -8 is not a level of the grid (never emitted by the quantizer)
                val = (float)q;
            } else {
                idx = (int)(nib & 7u);
                const float mag = GRID == UFP4_GRID_E1M2 ? 0.25f * (float)idx
                                                         : (idx < 2 ? 0.5f * (float)idx : (float)((2 + (idx & 1)) << ((idx >> 1) - 1)) * 0.5f);
                val = (nib & 8u) ? -mag : mag;
            }
            const float xp = v[i], xq = val * s, e = xq - xp;
            bxx = fmaf(xp, xp, bxx);
            bee = fmaf(e, e, bee);
            bxq = fmaf(xq, xp, bxq);
            hist += 1ull << (8 * idx);
            // level - t in grid units; a zero-scale block counts for the bucket ratio but has no t
            const float err = s > 0.0f ? fabsf(val) - fabsf(xp) * inv_s : 0.0f;
            lvl[idx][threadIdx.x] += err;
        }
        sxx += (double)bxx;
        see += (double)bee;
        sxq += (double)bxq;
#pragma unroll
        for (int k = 0; k < 8; ++k) cnt[k] += (int)((hist >> (8 * k)) & 0xFFu);
    }

    double vals[kDiagSums];
    vals[0] = sxx; vals[1] = see; vals[2] = sxq;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        vals[3 + k] = (double)cnt[k];
        vals[11 + k] = (double)lvl[k][threadIdx.x];
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int j = 0; j < kDiagSums; ++j) {
        double x = vals[j];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
        if (lane == 0) red[warp][j] = x;
    }
    __syncthreads();
    if (threadIdx.x < kDiagSums) {
        double x = 0.0;
        for (int w = 0; w < kDiagThreads / 32; ++w) x += red[w][threadIdx.x];
        P.partials[(int64_t)blockIdx.x * kDiagSums + threadIdx.x] = x;
    }
}

// out[j] = sum of the CTA partials: warp j adds them lane-strided, then across lanes in a fixed butterfly order.
__global__ void __launch_bounds__(32 * kDiagSums) diagnose_finish_kernel(const double *partials, int num_ctas, double *out) {
    const int j = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double x = 0.0;
    for (int c = lane; c < num_ctas; c += 32) x += partials[(int64_t)c * kDiagSums + j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
    if (lane == 0) out[j] = x;
}

}  // namespace ufp4

extern "C" size_t ufp4_diagnose_workspace_bytes(int64_t rows, int64_t cols) {
    (void)rows; (void)cols;
    return (size_t)2048 * ufp4::kDiagSums * sizeof(double);
}

extern "C" int ufp4_diagnose(const void *x, int64_t rows, int64_t cols, int64_t ld, const ufp4_qtensor *q_row, int rht_block,
                             uint64_t seed_rht, double *dev_out, void *workspace, size_t workspace_bytes, void *stream) {
    if (!x || !q_row || !q_row->codes || !q_row->scales || !dev_out || !workspace) return UFP4_ERR_NULL;
    if (rows < 1 || cols < 16 || cols % 16 != 0 || ld < cols || q_row->rows != rows || q_row->k != cols) return UFP4_ERR_SHAPE;
    if (rht_block != 0 && rht_block != 16 && rht_block != 32 && rht_block != 64 && rht_block != 128) return UFP4_ERR_UNSUPPORTED;
    if (rht_block > 16 && cols % rht_block != 0) return UFP4_ERR_SHAPE;
    if (q_row->grid < 0 || q_row->grid > 4) return UFP4_ERR_ENUM;
    if (q_row->scale_fmt == UFP4_SCALE_E4M3_TENSOR) return UFP4_ERR_UNSUPPORTED;
    if (!ufp4::aligned_to(x, 16) || (ld * 2) % 16 != 0 || !ufp4::aligned_to(q_row->codes, 8) || q_row->ld_codes_bytes % 8 != 0 ||
        !ufp4::aligned_to(dev_out, 8) || !ufp4::aligned_to(workspace, 8))
        return UFP4_ERR_ALIGN;
    if (workspace_bytes < ufp4_diagnose_workspace_bytes(rows, cols)) return UFP4_ERR_WORKSPACE;
    ufp4::DiagParams P = {};
    P.x = static_cast<const uint16_t *>(x);
    P.rows = rows; P.cols = cols; P.ld = ld;
    P.codes = static_cast<const uint8_t *>(q_row->codes);
    P.scales = static_cast<const float *>(q_row->scales);
    P.ldc = q_row->ld_codes_bytes; P.lds = q_row->ld_scales;
    P.grid = ufp4::codebook_of(q_row->grid); P.rht = rht_block != 0;
    P.xb = rht_block == 32 ? 1 : (rht_block == 64 ? 2 : (rht_block == 128 ? 3 : 0));
    P.norm = rht_block <= 16 ? 0.25f : (float)(1.0 / sqrt((double)rht_block));
    P.load256 = ufp4::aligned_to(x, 32) && ld % 16 == 0;
    ufp4_rht_signs(seed_rht, P.signs);
    P.partials = static_cast<double *>(workspace);
    const int64_t nblk = rows * (cols / 16);
    int64_t ctas = (nblk + ufp4::kDiagThreads - 1) / ufp4::kDiagThreads;
    if (ctas > 2048) ctas = 2048;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (P.grid == UFP4_GRID_INT4) ufp4::diagnose_kernel<UFP4_GRID_INT4><<<(unsigned)ctas, ufp4::kDiagThreads, 0, st>>>(P);
    else if (P.grid == UFP4_GRID_E1M2) ufp4::diagnose_kernel<UFP4_GRID_E1M2><<<(unsigned)ctas, ufp4::kDiagThreads, 0, st>>>(P);
    else ufp4::diagnose_kernel<UFP4_GRID_E2M1><<<(unsigned)ctas, ufp4::kDiagThreads, 0, st>>>(P);
    if (cudaGetLastError() != cudaSuccess) return UFP4_ERR_CUDA;
    ufp4::diagnose_finish_kernel<<<1, 32 * ufp4::kDiagSums, 0, st>>>(P.partials, (int)ctas, dev_out);
    return cudaGetLastError() == cudaSuccess ? UFP4_OK : UFP4_ERR_CUDA;
}

// The ratios of Sec. 3 from the 19 sums above (host arithmetic on 19 numbers, no launch).
extern "C" int ufp4_diagnose_ratios(const double *sums, double *out) {
    if (!sums || !out) return UFP4_ERR_NULL;
    const double sxx = sums[0];
    const double qnan = NAN;
    out[0] = sxx > 0.0 ? sums[2] / sxx : qnan;                       // alpha, Eq. 3
    out[1] = sxx > 0.0 ? sums[1] / sxx : qnan;                       // NMSE, Sec. 3.3
    double n = 0.0, ent = 0.0;
    for (int i = 0; i < 8; ++i) n += sums[3 + i];
    if (n > 0.0)
        for (int i = 0; i < 8; ++i) {
            const double p = sums[3 + i] / n;
            ent -= p * log(p + 1e-12);                              // Eq. 6: natural logarithm, eps = 1e-12
        }
    out[2] = exp(ent) / 8.0;                                        // B_eff over K = 8 magnitude buckets
    for (int i = 0; i < 8; ++i) out[3 + i] = sums[3 + i] > 0.0 ? sums[11 + i] / sums[3 + i] : qnan;
    return UFP4_OK;
}
