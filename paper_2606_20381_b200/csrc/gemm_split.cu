// Tensor-core path of the block-scaled 4-bit GEMM (Sec. 2.2: Y^ = Q_G(XH') Q_G(WH')^T) for arbitrary block scales, in
// particular the single-level FP32 scales of the paper's recipe (Table 1).
//
// With FP32 scales the dequantized value a = level * s has up to 27 significant bits, so it cannot ride in an 8-bit
// operand, and the scale product sA * sB differs for every (row, column, block), so it cannot be factored out of the
// product either.  Instead each operand is split, relative to a per-row power-of-two reference, into two FP16 numbers
//     a / ref = hi + 2^-11 lo        (hi = RN16(a / ref), lo = RN16(2^11 (a / ref - hi)): 22 significant bits)
// and the product is taken as  hi_a hi_b  +  2^-11 (hi_a lo_b + lo_a hi_b)  by three FP16 tensor-core MMAs per K step
// into two FP32 accumulators in tensor memory; the dropped lo_a lo_b term is 2^-22 of the product.  Every partial
// product is exact (11 x 11 bits); the relative error of a term is about 3 x 2^-23, far inside the 1e-5 bound.
// Two kernels:
//   1. decode_split_kernel: packed nibbles + scales -> hi and lo FP16 arrays [rows][K] and one FP32 reference per row
//      (caller's workspace); blocks more than 2^26 below the row's largest scale are flushed and reported.
//   2. gemm_split_kernel: the same warp-specialised, persistent CTA-pair design as the 8-bit kernel (TMA ring ->
//      tcgen05.mma cta_group::2 kind::f16 -> tcgen05.ld epilogue -> TMA store), with four operand tiles per stage and
//      the two accumulators filling tensor memory, so a tile's accumulators are read out before the next tile starts.
//
// One-piece variant (path FP16) for operands that both carry E4M3 block scales times a per-tensor FP32 scale (the
// NVFP4-style two-level hierarchy of Sec. 2.1's footnote): level * E4M3 value has at most 3 + 4 significant bits and
// lies in [2^-11, 3136], so it is exact in ONE FP16 number, needs no per-row reference and no exponent window, and the
// per-tensor scales multiply the result once in the epilogue.  The same two kernels run with the lo pieces left out:
// one MMA per K step, six operand stages instead of three and a double-buffered accumulator.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_bf16.h>
#include <stdlib.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tc.cuh"

namespace ufp4 {

constexpr int kSpK = 64;                              // K elements per stage: one 128-byte row of FP16
constexpr int kSpTile = kTM * kTK;                    // bytes of one 128-row operand tile of a stage (16 KB)
constexpr int kSpStageBytes = 4 * kSpTile;            // hi_a, lo_a, hi_b (this CTA's half), lo_b (this CTA's half)
constexpr int kSpStages = 3;
constexpr int kSpRing = kSpStages * kSpStageBytes;
// one-piece variant: hi_a and hi_b only, twice as many stages in the same ring
constexpr int kSp1StageBytes = 2 * kSpTile;
constexpr int kSp1Stages = 6;
static_assert(kSp1Stages * kSp1StageBytes == kSpRing, "both variants use the same ring");
constexpr int kSpMaxStages = 6;
constexpr int kSpEpiWarps = 8;
constexpr int kSpThreads = 64 + 32 * kSpEpiWarps;      // warp 0: TMA, warp 1: MMA + TMEM alloc, warps 2-9: epilogue
constexpr int kSpEpiBufBytes = 32 * 128;
constexpr int kSpOffEpi = kSpRing;
constexpr int kSpOffRefB = kSpOffEpi + kSpEpiWarps * kSpEpiBufBytes;
constexpr int kSpOffBars = kSpOffRefB + kTN * 4;         // one refB buffer: with it, a decode CTA (no shared memory, 64
                                                         // registers) fits on the SM beside this kernel's CTA
constexpr int kSpSmem = kSpOffBars + 256;
constexpr float kSpLoScale = 2048.0f;                 // 2^11
constexpr int kSpFlushExp = -15;                      // blocks whose normalised scale is below 2^-15 are flushed

// ------------------------------------------------------------------------------------------------------------------
// decode
// ------------------------------------------------------------------------------------------------------------------

struct SDecodeOperand {
    const uint8_t *codes;
    const void *scales;
    const float *tensor_scale;
    int64_t ldc, lds, rows;
    int grid, sfmt;
    __half *hi, *lo;    // [rows][K]
    float *ref;         // [rows]
};

struct SDecodeParams {
    SDecodeOperand op[2];   // A and B in one launch
    int64_t K;
    int64_t a_ctas;         // CTAs [0, a_ctas) work on A, the next ones on B
    int64_t tbl_cta;        // this CTA (if launched) lists the row tiles of a row-grouped product
    const int64_t *offsets; // row offsets of the groups (device), num_groups + 1 of them
    int num_groups;
    int2 *mtiles;           // (first row, group) of every 256-row tile, group by group
    int32_t *dev_status;
    int single;             // one-piece variant: both operands E4M3 x tensor scales; hi = level * E4M3 value, no lo
};

constexpr int kSDecodeThreads = 256;

__device__ __forceinline__ float split_scale_of(const SDecodeOperand &O, const void *srow, int kb, float ts) {
    if (O.sfmt == UFP4_SCALE_E4M3_TENSOR) {
        const uint8_t byte = static_cast<const uint8_t *>(srow)[kb];
        __half_raw hr = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)byte, __NV_E4M3);
        return __fmul_rn(ts, __half2float(*reinterpret_cast<__half *>(&hr)));
    }
    return __ldg(static_cast<const float *>(srow) + kb);
}

// 2^p for any p in [-252, 254] as the product of two normal floats.
__device__ __forceinline__ void pow2_factors(int p, float *f1, float *f2) {
    const int h = p / 2;
    *f1 = __uint_as_float((uint32_t)(h + 127) << 23);
    *f2 = __uint_as_float((uint32_t)(p - h + 127) << 23);
}

// A CTA decodes 256 / TPR rows with TPR threads (32..256) on each (more threads on long rows: no idle tail).
template <int TPR>
__global__ void __launch_bounds__(kSDecodeThreads) decode_split_kernel(const SDecodeParams P) {
    constexpr int kRowsPerCta = kSDecodeThreads / TPR;
    if ((int64_t)blockIdx.x == P.tbl_cta) {
        if (threadIdx.x == 0) {
            int n = 0;
            for (int g = 0; g < P.num_groups; ++g)
                for (int64_t m = P.offsets[g]; m < P.offsets[g + 1]; m += 2 * kTM) P.mtiles[n++] = make_int2((int)m, g);
        }
        return;
    }
    const bool is_b = (int64_t)blockIdx.x >= P.a_ctas;
    const SDecodeOperand &O = P.op[is_b ? 1 : 0];
    const int lane = threadIdx.x & 31;
    const int t = threadIdx.x % TPR;
    const int64_t row = ((int64_t)blockIdx.x - (is_b ? P.a_ctas : 0)) * kRowsPerCta + threadIdx.x / TPR;
    const bool active = row < O.rows;
    const int nkb = (int)(P.K >> 4);
    const float ts = O.sfmt == UFP4_SCALE_E4M3_TENSOR ? *O.tensor_scale : 1.0f;
    const int64_t r_safe = active ? row : 0;
    const void *srow = O.sfmt == UFP4_SCALE_E4M3_TENSOR
                           ? static_cast<const void *>(static_cast<const uint8_t *>(O.scales) + r_safe * O.lds)
                           : static_cast<const void *>(static_cast<const float *>(O.scales) + r_safe * O.lds);

    // largest block scale of the row (scales are non-negative: their bit patterns order like their values), eight loads
    // in flight per thread.  One or two warps per row: every warp scans the whole row (the repeats hit in cache) and no
    // barrier is needed.  Four or eight warps per row: a thread scans the scales of its own blocks only and the warps
    // combine through shared memory.
    uint32_t smax = 0u;
    if (P.single) {
        // one-piece variant: no row reference, nothing to scan
    } else if (TPR >= 128) {
        if (active) {
            int kb = t;
            for (; kb + 7 * TPR < nkb; kb += 8 * TPR) {
                float s[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) s[u] = split_scale_of(O, srow, kb + u * TPR, ts);
#pragma unroll
                for (int u = 0; u < 8; ++u) smax = max(smax, __float_as_uint(s[u]));
            }
            for (; kb < nkb; kb += TPR) smax = max(smax, __float_as_uint(split_scale_of(O, srow, kb, ts)));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) smax = max(smax, __shfl_xor_sync(0xFFFFFFFFu, smax, o));
        __shared__ uint32_t wmax[kSDecodeThreads / 32];
        if (lane == 0) wmax[threadIdx.x >> 5] = smax;
        __syncthreads();
        const int w0 = (threadIdx.x / TPR) * (TPR / 32);
#pragma unroll
        for (int i = 0; i < TPR / 32; ++i) smax = max(smax, wmax[w0 + i]);
    } else {
        if (active) {
            int kb = lane;
            for (; kb + 7 * 32 < nkb; kb += 8 * 32) {
                float s[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) s[u] = split_scale_of(O, srow, kb + u * 32, ts);
#pragma unroll
                for (int u = 0; u < 8; ++u) smax = max(smax, __float_as_uint(s[u]));
            }
            for (; kb < nkb; kb += 32) smax = max(smax, __float_as_uint(split_scale_of(O, srow, kb, ts)));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) smax = max(smax, __shfl_xor_sync(0xFFFFFFFFu, smax, o));
    }
    if (!active) return;

    // Reference 2^(e - 11), e the exponent of the largest scale: the largest normalised scale lies in [2^11, 2^12) and
    // |level| <= 7 (uniform grids; E2M1 values <= 6) keeps every |a / ref| below 2^15 < 65504.  The level units
    // (1/4 for E1M2) go into the normalisation factor.  A kept block has a normalised scale of at least 2^-15, so its
    // smallest non-zero |a / ref| is 2^-17, where the two pieces still carry it to 2^-36: 2^-19 relative.
    const int fexp = max((int)(smax >> 23), 1);              // biased exponent field (a denormal maximum counts as 2^-126)
    float n1, n2, r1, r2;
    pow2_factors(138 - fexp, &n1, &n2);                      // 2^(11 - e), e = fexp - 127
    pow2_factors(fexp - 138, &r1, &r2);
    const float unit = O.grid == UFP4_GRID_E1M2 ? 0.25f : (O.grid == UFP4_GRID_E2M1 ? 0.5f : 1.0f);
    n2 = __fmul_rn(n2, unit);
    // one-piece variant: the operand is level * E4M3 value itself (exact in FP16); the tensor scale is the "reference"
    const bool single = P.single != 0;
    const float ts_mul = single ? 1.0f : ts;
    if (single) {
        n1 = 1.0f;
        n2 = unit;
    }
    if (t == 0) O.ref[row] = single ? ts : (smax == 0u ? 1.0f : __fmul_rn(r1, r2));

    // Signed integer value of a nibble in its grid's unit (INT4: q, n >= 8 is n - 16; E1M2: +-(n & 7) quarters;
    // E2M1: +-{0,1,2,3,4,6,8,12} halves), offset by 16 so that it is a positive byte: a 16-entry table in four registers,
    // looked up four nibbles at a time by byte permutes (index n & 7 in each half, then the half that bit 3 names).
    const bool int4 = O.grid == UFP4_GRID_INT4;
    const uint32_t mag_lo = 0x03020100u, mag_hi = O.grid == UFP4_GRID_E2M1 ? 0x0C080604u : 0x07060504u;
    const uint32_t lutp_lo = mag_lo + 0x10101010u, lutp_hi = mag_hi + 0x10101010u;
    const uint32_t lutn_lo = int4 ? 0x0B0A0908u : 0x10101010u - mag_lo;      // INT4: n - 16 + 16 = n (8..11)
    const uint32_t lutn_hi = int4 ? 0x0F0E0D0Cu : 0x10101010u - mag_hi;
    const float bias = 8388608.0f + 16.0f;
    uint32_t flushed = 0u;
    const uint2 *cptr = reinterpret_cast<const uint2 *>(O.codes + row * O.ldc);
    uint4 *hptr = reinterpret_cast<uint4 *>(O.hi + row * P.K);
    uint4 *lptr = reinterpret_cast<uint4 *>(O.lo + row * P.K);
#pragma unroll 2
    for (int kb = t; kb < nkb; kb += TPR) {
        const float s = split_scale_of(O, srow, kb, ts_mul);
        uint2 cw = __ldg(cptr + kb);
        const float sn = __fmul_rn(__fmul_rn(s, n1), n2);           // normalised scale (with the level unit)
        const bool keep = single ? true : sn >= __uint_as_float((uint32_t)(kSpFlushExp + 127) << 23) * unit;
        flushed |= (keep || s == 0.0f) ? 0u : (cw.x | cw.y);
        cw.x = keep ? cw.x : 0u;
        cw.y = keep ? cw.y : 0u;
        const float snk = keep ? sn : 0.0f;
        uint32_t hw[8], lw[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t w = (q & 2 ? cw.y : cw.x) >> (q & 1 ? 16 : 0);
            const uint32_t sel = w & 0x7777u;
            const uint32_t pos = __byte_perm(lutp_lo, lutp_hi, sel), neg = __byte_perm(lutn_lo, lutn_hi, sel);
            const uint32_t vals = __byte_perm(pos, neg, ((w >> 1) & 0x4444u) | 0x3210u);   // four bytes: value + 16
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                // 2^23 + byte as a float's bits, minus (2^23 + 16): the signed integer value, exactly
                const float v0 = __fsub_rn(__uint_as_float(__byte_perm(vals, 0x4B000000u, 0x7440 + 2 * h)), bias);
                const float v1 = __fsub_rn(__uint_as_float(__byte_perm(vals, 0x4B000000u, 0x7441 + 2 * h)), bias);
                const float x0 = __fmul_rn(v0, snk), x1 = __fmul_rn(v1, snk);
                const __half2 hi2 = __floats2half2_rn(x0, x1);
                const float2 hf = __half22float2(hi2);
                const __half2 lo2 = __floats2half2_rn(__fmul_rn(__fsub_rn(x0, hf.x), kSpLoScale),
                                                      __fmul_rn(__fsub_rn(x1, hf.y), kSpLoScale));
                hw[2 * q + h] = *reinterpret_cast<const uint32_t *>(&hi2);
                lw[2 * q + h] = *reinterpret_cast<const uint32_t *>(&lo2);
            }
        }
        // one 32-byte store per block and piece (rows are 32-byte aligned: K is a multiple of 16)
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     :: "l"(hptr + 2 * kb), "r"(hw[0]), "r"(hw[1]), "r"(hw[2]), "r"(hw[3]), "r"(hw[4]), "r"(hw[5]), "r"(hw[6]), "r"(hw[7])
                     : "memory");
        if (!single)
            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                         :: "l"(lptr + 2 * kb), "r"(lw[0]), "r"(lw[1]), "r"(lw[2]), "r"(lw[3]), "r"(lw[4]), "r"(lw[5]), "r"(lw[6]), "r"(lw[7])
                         : "memory");
    }
    if (flushed != 0u && P.dev_status) atomicOr(P.dev_status, (int)UFP4_DEV_EXP_WINDOW);
}

// ------------------------------------------------------------------------------------------------------------------
// product
// ------------------------------------------------------------------------------------------------------------------

// kind::f16, A = B = FP16 (format code 0), D = F32, both K-major, M = 256 (CTA pair), N = 256.
constexpr uint32_t kSpInstrDesc = (1u << 4) | ((uint32_t)(kTN >> 3) << 17) | ((uint32_t)((kTM * 2) >> 4) << 24);

__device__ __forceinline__ void tc_mma_f16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p; }"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kSpInstrDesc), "r"(accumulate) : "memory");
}

// One pair of CTAs per 256 x 256 tile of C; the CTA of rank r holds rows [m0 + 128 r, +128) of both A pieces and rows
// [n0 + 128 r, +128) of both B pieces.  Accumulator 0 (columns 0..255 of tensor memory) takes hi_a hi_b, accumulator 1
// (columns 256..511) takes hi_a lo_b + lo_a hi_b.  Tiles, reduction ranges and expert rows come from tile_info: plain
// products, row-grouped products (256-row tiles laid out group by group) and reduction-grouped products alike.
// SINGLE: the one-piece variant (hi pieces only, one MMA per K step, the two accumulators used in turn).
template <bool SINGLE>
__global__ void __launch_bounds__(kSpThreads, 1)
gemm_split_kernel(const __grid_constant__ CUtensorMap tmAh, const __grid_constant__ CUtensorMap tmAl,
                  const __grid_constant__ CUtensorMap tmBh, const __grid_constant__ CUtensorMap tmBl,
                  const __grid_constant__ CUtensorMap tmC, const TcParams P) {
    constexpr int kStages = SINGLE ? kSp1Stages : kSpStages;
    constexpr int kStageBytes = SINGLE ? kSp1StageBytes : kSpStageBytes;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = smem_u32(smem);
    const uint32_t bars = base + kSpOffBars;
    const uint32_t full_bar = bars, empty_bar = bars + 8 * kSpMaxStages;
    const uint32_t tfull_bar = bars + 16 * kSpMaxStages, tempty_bar = tfull_bar + 16;    // two of each (SINGLE uses both)
    const uint32_t rb_bar = tempty_bar + 16;                // two barriers: refB written / refB read by everyone
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + kSpOffBars + 16 * kSpMaxStages + 48);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + kSpOffBars + 160);   // flag, poll limit

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)cluster_cta_rank();
    const int group_id = blockIdx.x / 2, num_groups_launched = gridDim.x / 2;
    const uint32_t lead_full_bar = map_to_cta(full_bar, 0);
    const uint32_t lead_tempty_bar = map_to_cta(tempty_bar, 0);
    const int nks_all = (int)((P.K + kSpK - 1) / kSpK);      // K steps of a tile that reduces over all of K

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar + 8 * s, 2);                  // one arrive.expect_tx per CTA of the pair
            mbar_init(empty_bar + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar + 8 * a, 1);
            mbar_init(tempty_bar + 8 * a, 2 * kSpEpiWarps);
        }
        mbar_init(rb_bar, 32 * kSpEpiWarps);
        mbar_init(rb_bar + 8, 32 * kSpEpiWarps);
        abort_flag[0] = (base & 1023u) ? 1u : 0u;           // the swizzled layouts below need the 1024-byte alignment
        abort_flag[1] = P.wait_limit ? P.wait_limit : kWaitLimit;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        tmem_alloc<2>(smem_u32((const void *)tmem_slot), 512);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                      // the peer's barriers exist before anything is signalled on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer: this CTA's 128 rows of hi_a, lo_a and its 128-row halves of hi_b, lo_b
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = group_id; ok && !P.skip_loads && tile < P.total_tiles; tile += num_groups_launched) {
                const TileInfo t = tile_info<2>(P, tile, rank);
                const int32_t m0 = (int32_t)t.m0, n0 = (int32_t)(t.b_row0 + t.n0) + rank * (kTN / 2);
                // tile_info counts the reduction in units of 128 elements; a K step here is 64
                const int ks0 = 2 * t.kb0, nks = P.mode == 2 ? 2 * t.nkb : nks_all;
                for (int ks = 0; ks < nks; ++ks) {
                    if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const int32_t kc = (ks0 + ks) * kSpK;
                    const uint32_t fb = lead_full_bar + 8 * stage, dst = base + stage * kStageBytes;
                    if (rank == 0) mbar_expect_tx(full_bar + 8 * stage, kStageBytes);
                    else mbar_expect_tx_cluster(fb, kStageBytes);
                    tma_load_2d_pair(dst, &tmAh, kc, m0, fb);
                    if (SINGLE) {
                        tma_load_2d_pair(dst + kSpTile, &tmBh, kc, n0, fb);
                    } else {
                        tma_load_2d_pair(dst + kSpTile, &tmAl, kc, m0, fb);
                        tma_load_2d_pair(dst + 2 * kSpTile, &tmBh, kc, n0, fb);
                        tma_load_2d_pair(dst + 3 * kSpTile, &tmBl, kc, n0, fb);
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // ---------------- MMA issuer (rank 0 of the pair)
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = group_id; ok && tile < P.total_tiles; tile += num_groups_launched) {
                const TileInfo t = tile_info<2>(P, tile, rank);
                const int nks = P.mode == 2 ? 2 * t.nkb : nks_all;
                if (nks == 0) continue;                       // empty group: the epilogue writes zeros
                if (!mbar_wait(tempty_bar + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * kTN;
                for (int ks = 0; ks < nks; ++ks) {
                    if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t st = base + stage * kStageBytes;
                    const uint64_t ah = umma_desc_sw128(st), al = umma_desc_sw128(st + kSpTile);
                    const uint64_t bh = umma_desc_sw128(st + (SINGLE ? 1 : 2) * kSpTile), bl = umma_desc_sw128(st + 3 * kSpTile);
#pragma unroll
                    for (int k = 0; k < kSpK / 16; ++k) {
                        // K = 16 FP16 elements = 32 bytes per instruction: +2 in the (address >> 4) field per step
                        const uint64_t o = (uint64_t)(2 * k);
                        const uint32_t first = (ks > 0 || k > 0) ? 1u : 0u;
                        tc_mma_f16_pair(d_tmem, ah + o, bh + o, first);
                        if (!SINGLE) {
                            tc_mma_f16_pair(tmem_base + kTN, ah + o, bl + o, first);
                            tc_mma_f16_pair(tmem_base + kTN, al + o, bh + o, 1u);
                        }
                    }
                    tc_commit<2>(empty_bar + 8 * stage);      // the stage is free (in both CTAs) once read
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit<2>(tfull_bar + 8 * acc);            // the tile's accumulator(s) complete (in both CTAs)
                if (SINGLE) {
                    acc ^= 1;
                    if (acc == 0) acc_phase ^= 1u;
                } else {
                    acc_phase ^= 1u;
                }
            }
        }
    } else {
        // ---------------- epilogue: (acc0 + 2^-11 acc1) x refA[m] refB[n] -> swizzled shared staging -> TMA store of C
        const int q = warp & 3;                            // TMEM lane quarter this warp may access
        const int half = (warp - 2) >> 2;                  // which four of the eight 32-column chunks this warp drains
        const int et = threadIdx.x - 64;
        uint8_t *buf = smem + kSpOffEpi + (warp - 2) * kSpEpiBufBytes;
        float *refb_s = reinterpret_cast<float *>(smem + kSpOffRefB);
        uint32_t acc_phase = 0, rb_written = 0, rb_read = 0;
        int acc = 0;
        bool first_tile = true;
        bool ok = true;
        for (int tile = group_id; ok && tile < P.total_tiles; tile += num_groups_launched) {
            const TileInfo t = tile_info<2>(P, tile, rank);
            const int64_t m0 = t.m0, n0 = t.n0;
            const bool has_k = P.mode == 2 ? t.nkb > 0 : true;
            const int64_t m_own = m0 + q * 32 + lane;
            const float ra = m_own < P.M ? P.refA[m_own] : 0.0f;
            {
                const int64_t n = n0 + et;
                // one buffer: wait until every epilogue thread has finished with the previous tile's values, write this
                // tile's, and wait until all of them are there (bounded, abortable waits instead of bar.sync)
                if (!first_tile) {
                    if (!mbar_wait_warp(rb_bar + 8, rb_read, abort_flag)) { ok = false; break; }
                    rb_read ^= 1u;
                }
                first_tile = false;
                refb_s[et] = n < P.N ? P.refB[t.b_row0 + n] : 0.0f;
                mbar_arrive(rb_bar);
                if (!mbar_wait_warp(rb_bar, rb_written, abort_flag)) { ok = false; break; }
                rb_written ^= 1u;
            }
            const float4 *rb4 = reinterpret_cast<const float4 *>(refb_s);
            if (has_k) {
                if (!mbar_wait_warp(tfull_bar + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
                tc_fence_after();
            }
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * kTN;
            const uint32_t lead_tempty = lead_tempty_bar + 8 * acc;
            if (has_k) {
                // which accumulator and barrier phase the next tile with a reduction uses
                if (SINGLE) {
                    acc ^= 1;
                    if (acc == 0) acc_phase ^= 1u;
                } else {
                    acc_phase ^= 1u;
                }
            }
            const int32_t c_row = (int32_t)(m0 + q * 32), c_grp = (int32_t)(t.c_row0 / (P.M > 0 ? P.M : 1));
            uint32_t v0[32], v1[32];
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const int c = 4 * half + cc;
                if (has_k) {
                    tc_ld32(taddr + (uint32_t)(c * 32), v0);
                    if (!SINGLE) tc_ld32(taddr + (uint32_t)(kTN + c * 32), v1);
                    tc_wait_ld();
                    if (SINGLE) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v1[j] = 0u;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v0[j] = v1[j] = 0u;
                }
                if (has_k && cc == 3) {
                    // every column of both accumulators has been read: hand them back to the MMA warp
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(lead_tempty);
                }
                const int64_t n_base = n0 + c * 32;
                if (n_base >= P.N || c_row >= t.row_end) continue;   // warp-uniform: the box is clipped or not this tile's
                float x[32];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float4 r = rb4[c * 8 + j];
                    const float rr[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        x[4 * j + u] = __fmaf_rn(__uint_as_float(v1[4 * j + u]), 1.0f / kSpLoScale, __uint_as_float(v0[4 * j + u])) * ra * rr[u];
                }
                if (n_base + 32 > P.N && P.n_unaligned) epi_store_box_plain(P, x, t.c_row0 + m_own, n_base, m_own < t.row_end);
                else epi_store_box_tma(P, &tmC, buf, lane, x, (int32_t)n_base, c_row, c_grp);
            }
            mbar_arrive(rb_bar + 8);                           // this thread has finished with the tile's refB values
        }
        epi_store_drain(lane);
    }
    tc_teardown<2>(abort_flag, P.dev_status, tmem_base, 512, warp);
}

// ------------------------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------------------------

static size_t sp_round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// hi and lo FP16 arrays of both operands, the two reference vectors, and the row-tile list of a row-grouped product
size_t gemm_split_workspace_bytes(int64_t a_rows, int64_t b_rows, int64_t K) {
    return 2 * sp_round_up((size_t)a_rows * K * 2, 256) + 2 * sp_round_up((size_t)b_rows * K * 2, 256) +
           sp_round_up((size_t)a_rows * 4, 256) + sp_round_up((size_t)b_rows * 4, 256) +
           sp_round_up((size_t)(a_rows / 128 + 2) * sizeof(int2), 256);
}

int gemm_split_kernel_launches() { return 2; }

// one-piece variant (path FP16): the hi arrays only
size_t gemm_fp16_workspace_bytes(int64_t a_rows, int64_t b_rows, int64_t K) {
    return sp_round_up((size_t)a_rows * K * 2, 256) + sp_round_up((size_t)b_rows * K * 2, 256) +
           sp_round_up((size_t)a_rows * 4, 256) + sp_round_up((size_t)b_rows * 4, 256) +
           sp_round_up((size_t)(a_rows / 128 + 2) * sizeof(int2), 256);
}

// level * E4M3 value is exact in FP16 (at most 7 significant bits, magnitudes in [2^-11, 3136]); the per-tensor FP32
// scales multiply the result.  Other scale formats need the two-piece split.
bool gemm_fp16_supported(const ufp4_qtensor *A, const ufp4_qtensor *B, int64_t M, int64_t N, int64_t K, int mode) {
    (void)mode;
    if (A->scale_fmt != UFP4_SCALE_E4M3_TENSOR || B->scale_fmt != UFP4_SCALE_E4M3_TENSOR) return false;
    if (K % 16 != 0 || M < 1 || N < 1) return false;
    if (A->rows > 0x3FFFFFFF || B->rows > 0x3FFFFFFF || K > 0x3FFFFFFF) return false;
    return true;
}

bool gemm_split_supported(const ufp4_qtensor *A, const ufp4_qtensor *B, int64_t M, int64_t N, int64_t K, int mode) {
    (void)mode;
    if (K % 16 != 0 || M < 1 || N < 1) return false;
    if (A->rows > 0x3FFFFFFF || B->rows > 0x3FFFFFFF || K > 0x3FFFFFFF) return false;
    return true;
}

static bool sp_make_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t K) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)kSpK, (cuuint32_t)kTM};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// single: the one-piece variant (path FP16); the caller has checked gemm_fp16_supported.
int gemm_split_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int mode,
                      int64_t M, int64_t N, int64_t K, const int64_t *offsets, const int64_t *host_offsets, int num_groups,
                      int64_t group_n, void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream,
                      bool single) {
    if (!aligned_to(workspace, 256)) return UFP4_ERR_ALIGN;
    if (workspace_bytes < (single ? gemm_fp16_workspace_bytes(A->rows, B->rows, K) : gemm_split_workspace_bytes(A->rows, B->rows, K)))
        return UFP4_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    const size_t a_bytes = sp_round_up((size_t)A->rows * K * 2, 256), b_bytes = sp_round_up((size_t)B->rows * K * 2, 256);
    const size_t np = single ? 1 : 2;                                   // pieces per operand
    __half *Ah = reinterpret_cast<__half *>(ws), *Al = single ? Ah : reinterpret_cast<__half *>(ws + a_bytes);
    __half *Bh = reinterpret_cast<__half *>(ws + np * a_bytes), *Bl = single ? Bh : reinterpret_cast<__half *>(ws + 2 * a_bytes + b_bytes);
    float *refA = reinterpret_cast<float *>(ws + np * a_bytes + np * b_bytes);
    float *refB = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(refA) + sp_round_up((size_t)A->rows * 4, 256));
    int2 *mtiles = reinterpret_cast<int2 *>(reinterpret_cast<uint8_t *>(refB) + sp_round_up((size_t)B->rows * 4, 256));
    // row-grouped product: 256-row tiles group by group (the decode launch lists them from the device offsets)
    int64_t row_tiles = 0;
    if (mode == 1)
        for (int g = 0; g < num_groups; ++g) row_tiles += (host_offsets[g + 1] - host_offsets[g] + 2 * kTM - 1) / (2 * kTM);

    SDecodeParams D = {};
    D.op[0] = SDecodeOperand{static_cast<const uint8_t *>(A->codes), A->scales, A->tensor_scale, A->ld_codes_bytes,
                             A->ld_scales, A->rows, codebook_of(A->grid), A->scale_fmt, Ah, Al, refA};
    D.op[1] = SDecodeOperand{static_cast<const uint8_t *>(B->codes), B->scales, B->tensor_scale, B->ld_codes_bytes,
                             B->ld_scales, B->rows, codebook_of(B->grid), B->scale_fmt, Bh, Bl, refB};
    D.K = K;
    D.dev_status = dev_status;
    D.single = single ? 1 : 0;
    int tpr = 32;           // a warp per row up to 8 blocks per thread, more threads on longer rows
    while (tpr < kSDecodeThreads && (K >> 4) >= (int64_t)16 * tpr) tpr *= 2;
    const int64_t rows_per_cta = kSDecodeThreads / tpr;
    D.a_ctas = (A->rows + rows_per_cta - 1) / rows_per_cta;
    D.tbl_cta = D.a_ctas + (B->rows + rows_per_cta - 1) / rows_per_cta;
    D.offsets = offsets; D.num_groups = num_groups; D.mtiles = mtiles;
    const int64_t decode_ctas = D.tbl_cta + (mode == 1 ? 1 : 0);
    if (decode_ctas > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    const unsigned dg = (unsigned)decode_ctas;
    if (tpr == 32) decode_split_kernel<32><<<dg, kSDecodeThreads, 0, st>>>(D);
    else if (tpr == 64) decode_split_kernel<64><<<dg, kSDecodeThreads, 0, st>>>(D);
    else if (tpr == 128) decode_split_kernel<128><<<dg, kSDecodeThreads, 0, st>>>(D);
    else decode_split_kernel<256><<<dg, kSDecodeThreads, 0, st>>>(D);
    if (cudaGetLastError() != cudaSuccess) return UFP4_ERR_CUDA;

    CUtensorMap tmAh, tmAl, tmBh, tmBl, tmC;
    if (!sp_make_map(&tmAh, Ah, A->rows, K) || !sp_make_map(&tmAl, Al, A->rows, K) || !sp_make_map(&tmBh, Bh, B->rows, K) ||
        !sp_make_map(&tmBl, Bl, B->rows, K))
        return UFP4_ERR_CUDA;
    {
        EncodeTiledFn fn = encode_tiled_fn();
        if (!fn) return UFP4_ERR_CUDA;
        // C as [groups][rows][cols] so that the TMA store clips at the end of each group's rows and at N
        const int64_t groups = mode == 2 ? num_groups : 1;
        const cuuint64_t es = c_is_bf16 ? 2 : 4;
        cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)M, (cuuint64_t)groups};
        cuuint64_t strides[2] = {(cuuint64_t)ldc * es, (cuuint64_t)M * (cuuint64_t)ldc * es};
        cuuint32_t box[3] = {32, 32, 1};
        cuuint32_t estr[3] = {1, 1, 1};
        if (fn(&tmC, c_is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, C, dims, strides, box,
               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, c_is_bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return UFP4_ERR_CUDA;
    }

    TcParams P = {};
    P.C = C; P.ldc = ldc; P.c_is_bf16 = c_is_bf16;
    P.M = M; P.N = N; P.K = K; P.mode = mode;
    P.offsets = offsets; P.num_groups = num_groups; P.group_n = group_n;
    P.refA = refA; P.refB = refB; P.dev_status = dev_status;
    P.mtiles = mtiles;
    P.mt = mode == 1 ? (int)row_tiles : (int)((M + 2 * kTM - 1) / (2 * kTM));
    P.nt = (int)((N + kTN - 1) / kTN);
    const int64_t total = (int64_t)P.mt * P.nt * (mode == 2 ? num_groups : 1);
    if (total < 1 || total > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    P.total_tiles = (int)total;
    P.n_unaligned = ((N * (c_is_bf16 ? 2 : 4)) % 16) != 0;
    P.wait_limit = debug_wait_limit();
    P.skip_loads = debug_skip_loads();

    static DeviceSetup slots[kMaxDevices];
    const DeviceSetup *dev = nullptr;
    const int rc_setup = device_setup(slots, [](int ordinal, DeviceSetup &d) -> int {
        UFP4_CUDA_OK(cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, ordinal));
        UFP4_CUDA_OK(cudaFuncSetAttribute(gemm_split_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSpSmem));
        UFP4_CUDA_OK(cudaFuncSetAttribute(gemm_split_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSpSmem));
        d.max_pairs = resident_pairs(gemm_split_kernel<false>, kSpThreads, kSpSmem, d.num_sms);
        return UFP4_OK;
    }, &dev);
    if (rc_setup != UFP4_OK) return rc_setup;
    const int max_pairs = dev->max_pairs;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(2 * (unsigned)(total < max_pairs ? total : max_pairs));
    cfg.blockDim = dim3(kSpThreads);
    cfg.dynamicSmemBytes = kSpSmem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t err = single ? cudaLaunchKernelEx(&cfg, gemm_split_kernel<true>, tmAh, tmAl, tmBh, tmBl, tmC, P)
                                   : cudaLaunchKernelEx(&cfg, gemm_split_kernel<false>, tmAh, tmAl, tmBh, tmBl, tmC, P);
    return err == cudaSuccess ? UFP4_OK : UFP4_ERR_CUDA;
}

}  // namespace ufp4
