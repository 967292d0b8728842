// Device-side pieces shared by the quantizer kernels (Sec. 2.1 quantizer and rounding rules, Sec. 2.2 RHT): packed FP32
// arithmetic, the Philox draw, block scale, rounding and nibble packing of one or two 16-element blocks.
#pragma once
#include <cuda_fp8.h>
#include <float.h>

#include "common.cuh"

namespace ufp4 {

constexpr int kTileR = 128;
constexpr int kTileC = 128;
constexpr int kThreads = 256;

// grid class of a kernel instance: the two uniform grids differ in the nibble encoding and in g_max
enum { GC_INT4 = 0, GC_E2M1 = 1, GC_E1M2 = 2 };

struct QuantParams {
    const uint16_t *x;
    int64_t rows, cols, ld, batch_stride;
    uint8_t *codes_row;
    void *scales_row;
    int64_t ldc_row, lds_row;
    uint8_t *codes_col;
    void *scales_col;
    int64_t ldc_col, lds_col;
    const float *ts_row, *ts_col;
    int32_t *dev_status;
    uint32_t sr_k0, sr_k1;
    uint32_t sr_keys[20];              // Philox round keys (k0, k1) of rounds 0..9 for seed_sr
    int do_row, do_col;
    int load256;                       // x and its row pitch are 32-byte aligned: 256-bit loads
    uint32_t sign_lo[8], sign_hi[8];   // row pass: bit 31 set where eps of element 2j / 2j+1 of a block is -1
    uint32_t sign_col[16];             // col pass: bit 31 set where eps of row i of a block is -1
    float e2m1_max;                    // E2M1 grids: g_max (6, or 4 / 2 for the range-restricted variants)
    float e2m1_d, e2m1_dr;             // E2M1 grids: the divisor of amax_v for the stored scale and RN(1 / divisor)
    // RHT blocks of 32 / 64 / 128 (quantize_wide_kernel only)
    uint32_t signs[4];                 // bit i of the 128: eps_i = -1
    int xb;                            // log2(rht_block / 16): butterfly stages that pair 16-element blocks
    int rotate;                        // 0: no RHT at all (rht_block 0)
    int b32;                           // 1 x 32 scale blocks: a block and its neighbour share the larger amax
    float rht_norm;                    // RN(1 / sqrt(rht_block))
};

// max(|a|, |b|, |c|), NaN-propagating (so that a NaN anywhere in a block reaches the non-finite check)
__device__ __forceinline__ float amax3(float a, float b, float c) {
    float d;
    asm("max.NaN.abs.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float amax2(float a, float b) {
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(fabsf(a)), "f"(fabsf(b)));
    return d;
}
__device__ __forceinline__ float amax16(const float (&v)[16]) {
    float m0 = amax3(v[0], v[1], v[2]), m1 = amax3(v[3], v[4], v[5]), m2 = amax3(v[6], v[7], v[8]);
    float m3 = amax3(v[9], v[10], v[11]), m4 = amax3(v[12], v[13], v[14]);
    return amax2(amax3(m0, m1, m2), amax3(m3, m4, v[15]));
}

// Packed FP32 pairs: one instruction performs the same IEEE operation on both halves.
// (explicit .rn PTX on register pairs; the pair is formed inside the asm so that no real instruction packs it)
#define UFP4_F32X2_OP(name, op)                                                                              \
    __device__ __forceinline__ float2 name(float2 a, float2 b) {                                             \
        float2 d;                                                                                            \
        asm("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; " op " rd, ra, rb; "       \
            "mov.b64 {%0, %1}, rd; }"                                                                        \
            : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));                                \
        return d;                                                                                            \
    }
UFP4_F32X2_OP(add2, "add.rn.f32x2")
UFP4_F32X2_OP(sub2, "sub.rn.f32x2")
UFP4_F32X2_OP(mul2, "mul.rn.f32x2")
#undef UFP4_F32X2_OP

// a * 1 + b: the same value as add2(a, b).  Used where a is itself a packed product: the assembler was seen to merge
// a packed multiply and a following packed add into one fused multiply-add (single rounding), which breaks the
// two-rounding definition y = RN(x * inv), q = rint(y); it cannot merge a multiply into this FMA's multiplicand.
__device__ __forceinline__ float2 add2_unfusable(float2 a, float2 b) {
    float2 d;
    asm("{ .reg .b64 ra, rb, rc, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mov.b64 rc, {%6, %6}; "
        "fma.rn.f32x2 rd, ra, rc, rb; mov.b64 {%0, %1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(1.0f));
    return d;
}

__device__ __forceinline__ float2 add2_ru(float2 a, float2 b) {
    float2 d;
    asm("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; add.rp.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{ .reg .b64 ra, rb, rc, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mov.b64 rc, {%6, %7}; "
        "fma.rn.f32x2 rd, ra, rb, rc; mov.b64 {%0, %1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}

// Philox4x32-10 of counter (b_lo, b_hi, variant, tag) with the ten round keys taken from the kernel parameters.
__device__ __forceinline__ void philox_block(const uint32_t (&keys)[20], uint64_t block_index, uint32_t variant,
                                             uint32_t (&out)[4]) {
    uint32_t c0 = (uint32_t)block_index, c1 = (uint32_t)(block_index >> 32), c2 = variant, c3 = kSrCounterTag;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t lo0 = 0xD2511F53u * c0, hi0 = __umulhi(0xD2511F53u, c0);
        const uint32_t lo1 = 0xCD9E8D57u * c2, hi1 = __umulhi(0xCD9E8D57u, c2);
        const uint32_t n0 = hi1 ^ c1 ^ keys[2 * r], n2 = hi0 ^ c3 ^ keys[2 * r + 1];
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Stochastic rounding of two normalised values onto the uniform grid, as packed FP32: returns 2^23 + 8 + q for both.
// rx, ry: the random words holding the elements' bytes, bx / by: which byte.  q = sign(y) ceil(|y| - thr) with
// thr = (r + 1/2) / 256.  One byte permute builds -T = -(128 + thr) exactly (exponent 2^7, r in mantissa bits 8..15, the
// half in bit 7).  d = RU(|y| - T) keeps the ceiling: an integer bound k - 128 >= |y| - T is representable, so rounding up
// cannot cross it.  RU(d + 2^23 + 136) = 2^23 + 8 + ceil(|y| - thr) (the sum is at least 2^23 + 7, where the spacing is
// 1), and |y| <= 7 (1 + 2^-23) keeps the magnitude at most 7 because thr >= 2^-9.
__device__ __forceinline__ float2 sr_round2(float2 y, uint32_t rx, int bx, uint32_t ry, int by) {
    const float2 nt = make_float2(__uint_as_float(__byte_perm(rx, 0xC3000080u, 0x7504 + (bx << 4))),
                                  __uint_as_float(__byte_perm(ry, 0xC3000080u, 0x7504 + (by << 4))));   // -(128 + thr)
    const float2 a = make_float2(fabsf(y.x), fabsf(y.y));
    const float2 m = add2_ru(add2_ru(a, nt), make_float2(8388744.0f, 8388744.0f));       // 2^23 + 8 + magnitude
    const float2 mag = sub2(m, make_float2(8388616.0f, 8388616.0f));
    const float2 sm = make_float2(__uint_as_float(__float_as_uint(mag.x) | (__float_as_uint(y.x) & 0x80000000u)),
                                  __uint_as_float(__float_as_uint(mag.y) | (__float_as_uint(y.y) & 0x80000000u)));
    return add2(sm, make_float2(8388616.0f, 8388616.0f));
}

// Butterfly stage of partner distance d (in pairs) over n pairs: (a, b) -> (a + b, a - b).
template <int N, int D>
__device__ __forceinline__ void butterfly_pairs(float2 (&p)[N]) {
#pragma unroll
    for (int j = 0; j < N; ++j) {
        if ((j & D) == 0) {
            float2 a = p[j], b = p[j + D];
            p[j] = add2(a, b);
            p[j + D] = sub2(a, b);
        }
    }
}

__device__ __forceinline__ uint32_t pack8_nibbles(const uint32_t (&t)[8]) {
    // sum_j t[j] * 16^j (mod 2^32) as a depth-3 multiply-add tree
    uint32_t p0 = t[1] * 16u + t[0], p1 = t[3] * 16u + t[2], p2 = t[5] * 16u + t[4], p3 = t[7] * 16u + t[6];
    uint32_t q0 = p1 * 256u + p0, q1 = p3 * 256u + p2;
    return q1 * 65536u + q0;
}

// Two's-complement nibbles -> sign|magnitude nibbles, eight at a time (magnitudes are at most 7).
__device__ __forceinline__ uint32_t twos_to_signmag(uint32_t w) {
    uint32_t m = (w & 0x88888888u) >> 3;
    return (w ^ (m * 7u)) + m;
}

// Clear the sign bit of nibbles whose magnitude is zero (zero is always encoded 0x0).
__device__ __forceinline__ uint32_t canonical_zero(uint32_t w) {
    uint32_t nz = ((w & 0x77777777u) + 0x77777777u) & 0x88888888u;
    return w & (nz | 0x77777777u);
}

// x / d for a constant d whose reciprocal c = RN(1/d) is given: q0 = RN(x c), r = x - d q0 (exact in an FMA),
// q = RN(q0 + r c).  Bit-identical to the IEEE division for d in {7, 1.75, 6} (checked over all 2^23 mantissas).
__device__ __forceinline__ float div_by_const(float x, float d, float c) {
    float q0 = __fmul_rn(x, c);
    float r = __fmaf_rn(-d, q0, x);
    return __fmaf_rn(r, c, q0);
}

// g / x for g in {7, 1.75, 6} and normal x with 2^-100 <= x <= 2^122: hardware reciprocal estimate and one residual
// correction of the quotient.  Bit-identical to the IEEE division on that domain (ufp4_selftest_division compares it
// with the IEEE division over all 2^23 mantissas: the few significant bits of g make a single correction enough);
// unlike the generic division it needs no range check or slow path.  Zero / tiny / non-finite x are the caller's.
__device__ __forceinline__ float const_over(float g, float x) {
    float r0;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(x));
    float q0 = __fmul_rn(g, r0);
    float e1 = __fmaf_rn(-x, q0, g);
    return __fmaf_rn(e1, r0, q0);
}

// Scale of one block from amax_v = max|v|, v = the values before the 1/4 of the RHT (v = x' without RHT).  Returns invq,
// the factor that takes v to code units (grid units for E2M1); *scale_bits receives the stored scale (FP32 bits or the
// E4M3 byte).  With x' = v / 4 exactly, amax = amax_v / 4, s = RN(amax / g) = RN(amax_v / (4 g)) and
// RN(g / amax) / 4 = RN(g / amax_v): the power-of-two factors commute with the roundings, so nothing is multiplied by
// 1/4 here.  The uniform grids' code unit (4 for E1M2: levels are quarters) folds in the same way: 4 RN(1.75 / a) = RN(7 / a).
template <int GC, int SFMT, bool RHT>
__device__ __forceinline__ float block_scale(float amax_v, const QuantParams &P, float tensor_scale, uint32_t *scale_bits,
                                             bool *nonfinite) {
    *nonfinite = !(amax_v <= FLT_MAX);
    bool zero = !(amax_v >= (RHT ? 0x1p-98f : 0x1p-100f));        // amax < 2^-100
    // g_max of the grid, seen from v: d = (4 if RHT) * g_max divides amax_v for the stored scale
    // (E2M1: g_max is a launch parameter, 6 or the 4 / 2 of the range-restricted variants, whose divisions are exact
    // scalings by a power of two)
    constexpr float gc = (GC == GC_E1M2) ? 1.75f : 7.0f;
    constexpr float dc = RHT ? 4.0f * gc : gc;
    constexpr float drc = 1.0f / dc;                             // RN(1 / d): 1/g scaled by a power of two
    const float d = (GC == GC_E2M1) ? P.e2m1_d : dc;
    const float dr = (GC == GC_E2M1) ? P.e2m1_dr : drc;
    const float gq = (GC == GC_E2M1) ? P.e2m1_max : 7.0f;       // g_max in code units
    float invq;
    uint32_t sbits;
    if (SFMT == UFP4_SCALE_FP32) {
        sbits = __float_as_uint(div_by_const(amax_v, d, dr));
        // the one-correction quotient is verified for g in {7, 1.75, 6} only: the restricted grids take the IEEE division
        invq = (GC == GC_E2M1 && gq != 6.0f) ? __fdiv_rn(gq, amax_v) : const_over(gq, amax_v);
    } else if (SFMT == UFP4_SCALE_POW2) {
        float z = div_by_const(amax_v, d, dr);
        sbits = (__float_as_uint(z) + 0x007FFFFFu) & 0x7F800000u;   // next power of two >= z
        // 1 / s, times the code unit, times 1/4 with the RHT: all in the exponent field
        constexpr uint32_t kOne = 0x7F000000u + ((GC == GC_E1M2) ? (2u << 23) : 0u) - (RHT ? (2u << 23) : 0u);
        invq = __uint_as_float(kOne - sbits);
    } else {
        float z = div_by_const(amax_v, d, dr);
        float u = __fdiv_rn(z, tensor_scale);
        uint32_t byte = zero ? 0u : (uint32_t)__nv_cvt_float_to_fp8(u, __NV_SATFINITE, __NV_E4M3);
        __half_raw hr = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)byte, __NV_E4M3);
        float dq = __half2float(*reinterpret_cast<__half *>(&hr));
        float s = __fmul_rn(tensor_scale, dq);
        if (byte == 0u || s == 0.0f) zero = true;
        const float to_code = (GC == GC_E1M2) ? 4.0f : 1.0f;
        invq = __fmul_rn(__fdiv_rn(1.0f, s), RHT ? 0.25f * to_code : to_code);   // power-of-two factors: exact
        sbits = byte;
    }
    if (zero) {
        invq = 0.0f;
        sbits = 0u;
    }
    *scale_bits = sbits;
    return invq;
}

// Rounding + packing of 16 values for every mode except the packed uniform-RTNE fast path.
template <int GC, int ROUND, int SFMT>
__device__ __forceinline__ uint2 round_pack16(const float (&v)[16], float invq, const QuantParams &P,
                                              uint64_t block_index, uint32_t variant) {
    uint32_t rnd[4] = {0u, 0u, 0u, 0u};
    if (ROUND == UFP4_ROUND_SR) {
        philox_block(P.sr_keys, block_index, variant, rnd);
    }
    uint32_t word[2];
#pragma unroll
    for (int hw = 0; hw < 2; ++hw) {
        uint32_t t[8];
        if (GC != GC_E2M1 && ROUND == UFP4_ROUND_RTNE) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float y = __fmul_rn(v[8 * hw + j], invq);
                if (SFMT == UFP4_SCALE_E4M3_TENSOR) y = fminf(fmaxf(y, -7.0f), 7.0f);
                // y + 8 + 2^23 rounds y to the nearest integer, ties to even; the low nibble is then q + 8
                t[j] = __float_as_uint(__fadd_rn(y, 8388616.0f));
            }
            uint32_t w = (pack8_nibbles(t) - 0xFB000000u) ^ 0x88888888u;   // strip the exponent bits, offset -> two's
            word[hw] = (GC == GC_E1M2) ? twos_to_signmag(w) : w;
        } else if (GC != GC_E2M1) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int e = 8 * hw + j;
                float y = __fmul_rn(v[e], invq);
                float a = fabsf(y);
                if (SFMT == UFP4_SCALE_E4M3_TENSOR) a = fminf(a, 7.0f);
                // round up iff frac(a) > thr = (r + 1/2) / 256, i.e. magnitude = ceil(a - thr); a - thr is exact in FP32
                // and a <= 7 (1 + 2^-23) keeps the result at most 7 because thr >= 2^-9
                uint32_t r = (rnd[e >> 2] >> (8 * (e & 3))) & 0xFFu;
                float thr = __fmaf_rn(__uint_as_float(0x4B000000u | r), 0x1p-8f, -(32768.0f - 0x1p-9f));
                float tf = __fadd_ru(__fsub_rn(a, thr), 8388608.0f);          // 2^23 + ceil(a - thr)
                float mag = __fsub_rn(tf, 8388608.0f);
                float sm = __uint_as_float(__float_as_uint(mag) | (__float_as_uint(y) & 0x80000000u));
                t[j] = __float_as_uint(__fadd_rn(sm, 8388616.0f));            // low nibble: q + 8
            }
            uint32_t w = (pack8_nibbles(t) - 0xFB000000u) ^ 0x88888888u;
            word[hw] = (GC == GC_E1M2) ? twos_to_signmag(w) : w;
        } else if (ROUND == UFP4_ROUND_RTNE) {
            uint32_t w = 0;
            // the conversion saturates at 6 by itself; a smaller g_max (range-restricted grids) or a block scale that
            // may undershoot amax / g_max (E4M3 scales) needs the clamp, |y| <= g_max (1 + 2^-23) otherwise
            const float gm = P.e2m1_max;
            const bool clamp = SFMT == UFP4_SCALE_E4M3_TENSOR || gm != 6.0f;      // uniform over the launch
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float y0 = __fmul_rn(v[8 * hw + 2 * j], invq), y1 = __fmul_rn(v[8 * hw + 2 * j + 1], invq);
                if (clamp) {
                    y0 = fminf(fmaxf(y0, -gm), gm);
                    y1 = fminf(fmaxf(y1, -gm), gm);
                }
                uint32_t b;
                asm("{ .reg .b8 t8; cvt.rn.satfinite.e2m1x2.f32 t8, %2, %1; cvt.u32.u8 %0, t8; }"
                    : "=r"(b) : "f"(y0), "f"(y1));
                w |= (b & 0xFFu) << (8 * j);
            }
            word[hw] = canonical_zero(w);
        } else {
            // E2M1, SR.  The level spacing is 2^(k-1) on segment k: [0, 2), [2, 4), [4, 6].  In units of its segment's
            // spacing a value rounds like the uniform grid: magnitude = ceil(a_s - thr), thr = (r + 1/2) / 256, and the
            // level index is that integer + 2 k (segment 0: 0..4, segment 1: 2..4 -> 4..6, segment 2: 2..3 -> 6..7).
            // -(128 + thr) comes from one byte permute and the two additions round up, as in sr_round2: the ceiling is
            // kept because an integer bound is representable, and the offset 8 keeps the sum where the spacing is 1.
            const float gm = P.e2m1_max;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int e = 8 * hw + j;
                const float y = __fmul_rn(v[e], invq);
                const uint32_t ab = __float_as_uint(fminf(fabsf(y), gm));
                // segment from the exponent field ([0,2) -> 0, [2,4) -> 1, [4,8) -> 2); the scaling a * 2^(1 - k) is an
                // exponent-field addition (a zero or tiny a becomes some tiny positive number: level 0 all the same)
                const uint32_t k = (uint32_t)max((int)(ab >> 23) - 127, 0);
                const float as = __uint_as_float(ab + 0x00800000u - (k << 23));
                const float nt = __uint_as_float(__byte_perm(rnd[e >> 2], 0xC3000080u, 0x7504 + ((e & 3) << 4)));
                const float m = __fadd_ru(__fadd_ru(as, nt), 8388744.0f);              // 2^23 + 8 + ceil(a_s - thr)
                const uint32_t idx = (__float_as_uint(m) & 7u) + 2u * k;
                t[j] = idx ? (idx | ((__float_as_uint(y) >> 28) & 8u)) : 0u;
            }
            word[hw] = pack8_nibbles(t);
        }
    }
    return make_uint2(word[0], word[1]);
}

// Packed fast path (uniform grid, RTNE, no clamp): eight pairs -> two code words.  sel 0 packs the .x halves of 16
// pairs, sel 1 the .y halves (col pass: two columns at once); the row pass packs both halves of 8 pairs.
template <int GC>
__device__ __forceinline__ uint32_t finish_word(uint32_t packed) {
    uint32_t w = (packed - 0xFB000000u) ^ 0x88888888u;   // strip the exponent bits of 2^23 + 8 + q, offset -> two's
    return (GC == GC_E1M2) ? twos_to_signmag(w) : w;
}

__device__ __forceinline__ void store_scale(void *base, int64_t index, uint32_t bits, bool byte_scale) {
    if (byte_scale) reinterpret_cast<uint8_t *>(base)[index] = (uint8_t)bits;
    else reinterpret_cast<uint32_t *>(base)[index] = bits;
}

// Two 16-element blocks at once: pair i = (element i of block 0, element i of block 1), RHT signs already applied.
// Every butterfly stage is then pair-to-pair, i.e. one packed instruction per two additions.
// Rounding and packing of two blocks held as pairs, given their factors inv0 / inv1 (from block_scale).
template <int GC, int ROUND, int SFMT>
__device__ __forceinline__ void round_pair(const float2 (&q)[16], float inv0, float inv1, const QuantParams &P,
                                           uint64_t bidx0, uint64_t bidx1, uint32_t variant, uint2 *c0, uint2 *c1) {
    constexpr bool kFast = (GC != GC_E2M1 && ROUND == UFP4_ROUND_RTNE && SFMT != UFP4_SCALE_E4M3_TENSOR);
    if (kFast) {
        const float2 inv2 = make_float2(inv0, inv1);
        const float2 magic2 = make_float2(8388616.0f, 8388616.0f);
        uint32_t tx[16], ty[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            float2 t = add2_unfusable(mul2(q[i], inv2), magic2);
            tx[i] = __float_as_uint(t.x);
            ty[i] = __float_as_uint(t.y);
        }
        const uint32_t a0[8] = {tx[0], tx[1], tx[2], tx[3], tx[4], tx[5], tx[6], tx[7]};
        const uint32_t a1[8] = {tx[8], tx[9], tx[10], tx[11], tx[12], tx[13], tx[14], tx[15]};
        const uint32_t b0[8] = {ty[0], ty[1], ty[2], ty[3], ty[4], ty[5], ty[6], ty[7]};
        const uint32_t b1[8] = {ty[8], ty[9], ty[10], ty[11], ty[12], ty[13], ty[14], ty[15]};
        *c0 = make_uint2(finish_word<GC>(pack8_nibbles(a0)), finish_word<GC>(pack8_nibbles(a1)));
        *c1 = make_uint2(finish_word<GC>(pack8_nibbles(b0)), finish_word<GC>(pack8_nibbles(b1)));
    } else if (GC != GC_E2M1 && ROUND == UFP4_ROUND_SR && SFMT != UFP4_SCALE_E4M3_TENSOR) {
        uint32_t r0[4], r1[4];
        philox_block(P.sr_keys, bidx0, variant, r0);
        philox_block(P.sr_keys, bidx1, variant, r1);
        const float2 inv2 = make_float2(inv0, inv1);
        uint32_t tx[16], ty[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            float2 t = sr_round2(mul2(q[i], inv2), r0[i >> 2], i & 3, r1[i >> 2], i & 3);
            tx[i] = __float_as_uint(t.x);
            ty[i] = __float_as_uint(t.y);
        }
        const uint32_t a0[8] = {tx[0], tx[1], tx[2], tx[3], tx[4], tx[5], tx[6], tx[7]};
        const uint32_t a1[8] = {tx[8], tx[9], tx[10], tx[11], tx[12], tx[13], tx[14], tx[15]};
        const uint32_t b0[8] = {ty[0], ty[1], ty[2], ty[3], ty[4], ty[5], ty[6], ty[7]};
        const uint32_t b1[8] = {ty[8], ty[9], ty[10], ty[11], ty[12], ty[13], ty[14], ty[15]};
        *c0 = make_uint2(finish_word<GC>(pack8_nibbles(a0)), finish_word<GC>(pack8_nibbles(a1)));
        *c1 = make_uint2(finish_word<GC>(pack8_nibbles(b0)), finish_word<GC>(pack8_nibbles(b1)));
    } else if (GC == GC_E2M1 && ROUND == UFP4_ROUND_SR && SFMT != UFP4_SCALE_E4M3_TENSOR) {
        // E2M1 SR on pairs, the arithmetic of round_pack16's E2M1 SR branch: the segment k of a magnitude (level
        // spacing 2^(k-1)) comes from its exponent field, the scaling to segment units is an exponent-field addition.
        uint32_t r0[4], r1[4];
        philox_block(P.sr_keys, bidx0, variant, r0);
        philox_block(P.sr_keys, bidx1, variant, r1);
        const float2 inv2 = make_float2(inv0, inv1);
        const float gm = P.e2m1_max;
        uint32_t tx[16], ty[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float2 y = mul2(q[i], inv2);
            const uint32_t ax = __float_as_uint(fminf(fabsf(y.x), gm)), ay = __float_as_uint(fminf(fabsf(y.y), gm));
            const int kx = max((int)(ax >> 23) - 127, 0), ky = max((int)(ay >> 23) - 127, 0);     // 0, 1, 2
            // a * 2^(1 - k); a zero or tiny a becomes some tiny positive number, which rounds to level 0 all the same
            const float2 as = make_float2(__uint_as_float(ax + 0x00800000u - ((uint32_t)kx << 23)),
                                          __uint_as_float(ay + 0x00800000u - ((uint32_t)ky << 23)));
            const float2 nt = make_float2(__uint_as_float(__byte_perm(r0[i >> 2], 0xC3000080u, 0x7504 + ((i & 3) << 4))),
                                          __uint_as_float(__byte_perm(r1[i >> 2], 0xC3000080u, 0x7504 + ((i & 3) << 4))));
            const float2 m = add2_ru(add2_ru(as, nt), make_float2(8388744.0f, 8388744.0f));   // 2^23 + 8 + ceil(a_s - thr)
            tx[i] = ((__float_as_uint(m.x) & 7u) + 2u * (uint32_t)kx) | ((__float_as_uint(y.x) >> 28) & 8u);
            ty[i] = ((__float_as_uint(m.y) & 7u) + 2u * (uint32_t)ky) | ((__float_as_uint(y.y) >> 28) & 8u);
        }
        const uint32_t a0[8] = {tx[0], tx[1], tx[2], tx[3], tx[4], tx[5], tx[6], tx[7]};
        const uint32_t a1[8] = {tx[8], tx[9], tx[10], tx[11], tx[12], tx[13], tx[14], tx[15]};
        const uint32_t b0[8] = {ty[0], ty[1], ty[2], ty[3], ty[4], ty[5], ty[6], ty[7]};
        const uint32_t b1[8] = {ty[8], ty[9], ty[10], ty[11], ty[12], ty[13], ty[14], ty[15]};
        *c0 = make_uint2(canonical_zero(pack8_nibbles(a0)), canonical_zero(pack8_nibbles(a1)));
        *c1 = make_uint2(canonical_zero(pack8_nibbles(b0)), canonical_zero(pack8_nibbles(b1)));
    } else {
        float v0[16], v1[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            v0[i] = q[i].x;
            v1[i] = q[i].y;
        }
        *c0 = round_pack16<GC, ROUND, SFMT>(v0, inv0, P, bidx0, variant);
        *c1 = round_pack16<GC, ROUND, SFMT>(v1, inv1, P, bidx1, variant);
    }
}

template <int GC, int ROUND, int SFMT, bool RHT>
__device__ __forceinline__ void quantize_pair(float2 (&q)[16], const QuantParams &P, float tensor_scale, uint64_t bidx0,
                                              uint64_t bidx1, uint32_t variant, uint2 *c0, uint2 *c1, uint32_t *s0,
                                              uint32_t *s1, bool *nonfinite) {
    if (RHT) {
        butterfly_pairs<16, 1>(q);
        butterfly_pairs<16, 2>(q);
        butterfly_pairs<16, 4>(q);
        butterfly_pairs<16, 8>(q);
    }
    float v0[16], v1[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        v0[i] = q[i].x;
        v1[i] = q[i].y;
    }
    bool nf0, nf1;
    const float inv0 = block_scale<GC, SFMT, RHT>(amax16(v0), P, tensor_scale, s0, &nf0);
    const float inv1 = block_scale<GC, SFMT, RHT>(amax16(v1), P, tensor_scale, s1, &nf1);
    *nonfinite |= nf0 | nf1;
    round_pair<GC, ROUND, SFMT>(q, inv0, inv1, P, bidx0, bidx1, variant, c0, c1);
}

// Launchers of the kernels that live in files of their own (gc: grid class, GC_*).
cudaError_t launch_quantize_wide(int gc, int rounding, int sfmt, dim3 grid, cudaStream_t st, const QuantParams &P);

}  // namespace ufp4
