// Fused RHT + blockwise quantizer for RHT blocks of 32 / 64 / 128 elements and for 1 x 32 scale blocks (App. B's block-size
// search; Sec. 2.1's footnote on MXFP4): the plain kernel beside the benchmarked 16-point one.
#include "quantize_core.cuh"

namespace ufp4 {

// ------------------------------------------------------------------------------------------------------------------
// RHT blocks of 32 / 64 / 128 elements (the block sizes App. B searched beside the selected 16).  H_n = H_(n/16) (x) H_16:
// the stages h = 1..8 run inside the thread that holds a 16-element block, the stages h = 16, 32, 64 pair whole
// 16-element blocks, which the eight neighbouring lanes of a tile row (row pass) or of a tile column (col pass) hold, so
// they are register exchanges between lanes.  The result is scaled by RN(1 / sqrt(n)) explicitly (not a power of two for
// n = 32, 128) and quantized like an unrotated block.  A plain kernel: this variant is not on the benchmarked path.
// ------------------------------------------------------------------------------------------------------------------
// The 16 sign bits of the 16-element block at place blk of its RHT block.
__device__ __forceinline__ uint32_t wide_sign_bits(const QuantParams &P, int blk) {
    const int j = blk & ((1 << P.xb) - 1);
    return P.rotate ? (P.signs[j >> 1] >> (16 * (j & 1))) & 0xFFFFu : 0u;
}

// q[i] = (element i of block 0, element i of block 1): two 16-element blocks that sit at the same place of their RHT
// blocks, signs already applied (on the raw BF16 words), rotated together with packed instructions.
__device__ __forceinline__ void wide_rotate2(float2 (&q)[16], const QuantParams &P, int blk) {
    if (!P.rotate) return;                                          // uniform over the launch
    butterfly_pairs<16, 1>(q);
    butterfly_pairs<16, 2>(q);
    butterfly_pairs<16, 4>(q);
    butterfly_pairs<16, 8>(q);
    for (int s = 0; s < P.xb; ++s) {
        const int m = 1 << s;
        const bool upper = (blk & m) != 0;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float2 o = make_float2(__shfl_xor_sync(0xFFFFFFFFu, q[i].x, m), __shfl_xor_sync(0xFFFFFFFFu, q[i].y, m));
            q[i] = upper ? sub2(o, q[i]) : add2(q[i], o);
        }
    }
    const float2 n2 = make_float2(P.rht_norm, P.rht_norm);
#pragma unroll
    for (int i = 0; i < 16; ++i) q[i] = mul2(q[i], n2);
}

// Scale, round and pack the two rotated blocks of q; in0 / in1: the block lies inside the matrix (the exchanges above
// and the amax exchange here are done by every lane).
template <int GC, int ROUND, int SFMT>
__device__ __forceinline__ void wide_finish2(const float2 (&q)[16], const QuantParams &P, float ts, bool in0, bool in1,
                                             uint64_t bidx0, uint64_t bidx1, uint32_t variant, uint8_t *codes0,
                                             uint8_t *codes1, void *scales, int64_t sidx0, int64_t sidx1,
                                             bool *nonfinite) {
    float v0[16], v1[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        v0[i] = q[i].x;
        v1[i] = q[i].y;
    }
    float a0 = amax16(v0), a1 = amax16(v1);
    if (P.b32) {
        a0 = amax2(a0, __shfl_xor_sync(0xFFFFFFFFu, a0, 1));
        a1 = amax2(a1, __shfl_xor_sync(0xFFFFFFFFu, a1, 1));
    }
    const bool byte_scale = (SFMT == UFP4_SCALE_E4M3_TENSOR);
    uint32_t sb0, sb1;
    bool nf0, nf1;
    const float inv0 = block_scale<GC, SFMT, false>(a0, P, ts, &sb0, &nf0);
    const float inv1 = block_scale<GC, SFMT, false>(a1, P, ts, &sb1, &nf1);
    uint2 c0, c1;
    round_pair<GC, ROUND, SFMT>(q, inv0, inv1, P, bidx0, bidx1, variant, &c0, &c1);
    if (in0) {
        *nonfinite |= nf0;
        *reinterpret_cast<uint2 *>(codes0) = c0;
        store_scale(scales, sidx0, sb0, byte_scale);
    }
    if (in1) {
        *nonfinite |= nf1;
        *reinterpret_cast<uint2 *>(codes1) = c1;
        store_scale(scales, sidx1, sb1, byte_scale);
    }
}

template <int GC, int ROUND, int SFMT>
__global__ void __launch_bounds__(kThreads) quantize_wide_kernel(const QuantParams P) {
    // raw BF16 pairs; the 16-byte chunk c of tile row r sits at chunk c ^ ((r >> 4) & 7), so that the col pass, whose
    // eight lanes of a column pair read rows 16 apart, hits eight different bank groups
    __shared__ __align__(16) uint32_t tile[kTileR][kTileC / 2];
    const int tid = threadIdx.x;
    const int64_t e = blockIdx.z;
    const int64_t row0 = (int64_t)blockIdx.y * kTileR, col0 = (int64_t)blockIdx.x * kTileC;
    const bool byte_scale = (SFMT == UFP4_SCALE_E4M3_TENSOR);
    const float ts_row = (byte_scale && P.do_row) ? *P.ts_row : 1.0f;
    const float ts_col = (byte_scale && P.do_col) ? *P.ts_col : 1.0f;
    bool any_nonfinite = false;

    // ---- row pass: thread t owns 16-element block b = t & 7 of rows (t >> 3) + 32 it; two rows at a time
    const int ra = tid >> 3, ba = tid & 7;
    const int64_t gca = col0 + 16 * ba;
#pragma unroll 1
    for (int it = 0; it < 4; it += 2) {
        uint4 d[2][2];
        bool in[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int rl = ra + 32 * (it + h);
            in[h] = gca < P.cols && row0 + rl < P.rows;
            d[h][0] = make_uint4(0, 0, 0, 0);
            d[h][1] = d[h][0];
            if (in[h]) {
                const uint4 *s4 = reinterpret_cast<const uint4 *>(P.x + e * P.batch_stride + (row0 + rl) * P.ld + gca);
                d[h][0] = __ldg(s4);
                d[h][1] = __ldg(s4 + 1);
            }
            if (P.do_col) {
                uint4 *dst = reinterpret_cast<uint4 *>(&tile[rl][0]);
                const int sw = (rl >> 4) & 7;
                dst[(2 * ba) ^ sw] = d[h][0];
                dst[(2 * ba + 1) ^ sw] = d[h][1];
            }
        }
        if (P.do_row) {                                             // uniform: every lane takes part in the exchanges
            const uint32_t w0[8] = {d[0][0].x, d[0][0].y, d[0][0].z, d[0][0].w, d[0][1].x, d[0][1].y, d[0][1].z, d[0][1].w};
            const uint32_t w1[8] = {d[1][0].x, d[1][0].y, d[1][0].z, d[1][0].w, d[1][1].x, d[1][1].y, d[1][1].z, d[1][1].w};
            const uint32_t sb = wide_sign_bits(P, ba);
            float2 q[16];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                // BF16 sign bits of elements 2j (bit 15) and 2j + 1 (bit 31) of the raw word, for both rows
                const uint32_t sg = (((sb >> (2 * j)) & 1u) << 15) | (((sb >> (2 * j + 1)) & 1u) << 31);
                const uint32_t x0 = w0[j] ^ sg, x1 = w1[j] ^ sg;
                q[2 * j] = make_float2(__uint_as_float(x0 << 16), __uint_as_float(x1 << 16));
                q[2 * j + 1] = make_float2(__uint_as_float(x0 & 0xFFFF0000u), __uint_as_float(x1 & 0xFFFF0000u));
            }
            wide_rotate2(q, P, ba);
            const int64_t r0 = e * P.rows + row0 + ra + 32 * it, r1 = r0 + 32;
            const int64_t nb = P.cols >> 4, kb = gca >> 4;
            wide_finish2<GC, ROUND, SFMT>(q, P, ts_row, in[0], in[1], (uint64_t)(r0 * nb + kb), (uint64_t)(r1 * nb + kb), 0u,
                                          P.codes_row + r0 * P.ldc_row + (gca >> 1), P.codes_row + r1 * P.ldc_row + (gca >> 1),
                                          P.scales_row, r0 * P.lds_row + kb, r1 * P.lds_row + kb, &any_nonfinite);
        }
    }

    if (P.do_col) {
        __syncthreads();
        // ---- col pass: lane l of warp w owns the 16-row block rb = l & 7 of columns 2 cp, 2 cp + 1,
        // cp = 32 it + 4 w + (l >> 3)
        const int rb = tid & 7, cq = (tid >> 3) & 3, wp = tid >> 5;
        const int64_t nrb = P.rows >> 4, grb = (row0 >> 4) + rb;
#pragma unroll 1
        for (int it = 0; it < 2; ++it) {
            const int cp = 32 * it + 4 * wp + cq;
            const int64_t gc = col0 + 2 * cp;
            const bool in = gc < P.cols && grb < nrb;              // columns come in pairs: cols is a multiple of 16
            const int pos = (((cp >> 2) ^ rb) << 2) | (cp & 3);
            const uint32_t sb = wide_sign_bits(P, rb);
            float2 q[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                // row i of the block carries one sign for both columns of the word
                const uint32_t ww = tile[16 * rb + i][pos] ^ (((sb >> i) & 1u) * 0x80008000u);
                q[i] = make_float2(__uint_as_float(ww << 16), __uint_as_float(ww & 0xFFFF0000u));
            }
            wide_rotate2(q, P, rb);
            const int64_t c0 = e * P.cols + gc, c1 = c0 + 1;
            wide_finish2<GC, ROUND, SFMT>(q, P, ts_col, in, in, (uint64_t)(c0 * nrb + grb), (uint64_t)(c1 * nrb + grb), 1u,
                                          P.codes_col + c0 * P.ldc_col + grb * 8, P.codes_col + c1 * P.ldc_col + grb * 8,
                                          P.scales_col, c0 * P.lds_col + grb, c1 * P.lds_col + grb, &any_nonfinite);
        }
    }
    if (any_nonfinite && P.dev_status) atomicOr(P.dev_status, (int)UFP4_DEV_NONFINITE);
}

template <int GC, int ROUND>
static cudaError_t launch_wide(int sfmt, dim3 grid, cudaStream_t st, const QuantParams &P) {
    switch (sfmt) {
        case UFP4_SCALE_FP32: quantize_wide_kernel<GC, ROUND, UFP4_SCALE_FP32><<<grid, kThreads, 0, st>>>(P); break;
        case UFP4_SCALE_POW2:
        case UFP4_SCALE_E8M0_B32: quantize_wide_kernel<GC, ROUND, UFP4_SCALE_POW2><<<grid, kThreads, 0, st>>>(P); break;
        default: quantize_wide_kernel<GC, ROUND, UFP4_SCALE_E4M3_TENSOR><<<grid, kThreads, 0, st>>>(P); break;
    }
    return cudaGetLastError();
}

cudaError_t launch_quantize_wide(int gc, int rounding, int sfmt, dim3 grid, cudaStream_t st, const QuantParams &P) {
    const bool sr = rounding == UFP4_ROUND_SR;
    if (gc == GC_E2M1) return sr ? launch_wide<GC_E2M1, UFP4_ROUND_SR>(sfmt, grid, st, P) : launch_wide<GC_E2M1, UFP4_ROUND_RTNE>(sfmt, grid, st, P);
    if (gc == GC_E1M2) return sr ? launch_wide<GC_E1M2, UFP4_ROUND_SR>(sfmt, grid, st, P) : launch_wide<GC_E1M2, UFP4_ROUND_RTNE>(sfmt, grid, st, P);
    return sr ? launch_wide<GC_INT4, UFP4_ROUND_SR>(sfmt, grid, st, P) : launch_wide<GC_INT4, UFP4_ROUND_RTNE>(sfmt, grid, st, P);
}

}  // namespace ufp4
