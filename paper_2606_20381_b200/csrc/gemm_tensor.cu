// Tensor-core path of the block-scaled 4-bit GEMM (Sec. 2.2: Y^ = Q_G(XH') Q_G(WH')^T) for power-of-two block scales.
//
// B200's tensor cores have no uniform 4-bit element type (the paper's premise, Sec. 1 and Sec. 6), so the product is
// computed exactly on 8-bit floating-point operands instead: with a power-of-two block scale 2^e, the dequantized
// value q * 2^e (|q| <= 7, or 2*value <= 12 for the E2M1 grid: at most 3 significant bits) is exactly representable
// in E5M2 once a per-row reference exponent is factored out.  Two kernels:
//   1. decode_rows_kernel: packed nibbles + scales  ->  E5M2 bytes [rows][K] and one FP32 reference scale per row
//      (caller's workspace); blocks more than 2^26 below the row's largest block are flushed and reported.
//   2. gemm_tc_kernel: persistent, warp-specialised.  One thread issues TMA tile loads (128B-swizzled ring), one thread
//      issues tcgen05.mma kind::f8f6f4 (N256 x K32; M128 per CTA, or M256 on a CTA pair with cta_group::2) into a
//      double-buffered FP32 accumulator in tensor memory, eight warps drain accumulators with tcgen05.ld, apply
//      refA[m] * refB[n] and hand 32 x 32 boxes of C to TMA stores.
// Every product q_a 2^ea * q_b 2^eb is exact; accumulation is the tensor core's FP32.
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdio.h>
#include <stdlib.h>

#include "common.cuh"
#include "ptx.cuh"
#include "quantize_core.cuh"
#include "tc.cuh"

namespace ufp4 {

constexpr int kUmmaK = 32;                          // K of one kind::f8f6f4 instruction
constexpr int kAStage = kTM * kTK;
constexpr int kEpiWarps = 8;                        // two per TMEM lane quarter, each taking half of the columns
constexpr int kTcThreads = 64 + 32 * kEpiWarps;      // warp 0: TMA, warp 1: MMA + TMEM alloc, warps 2-9: epilogue
constexpr int kBarrierBytes = 256;
constexpr int kEpiBufBytes = 32 * 128;              // one staged 32-row x 32-column chunk (FP32; BF16 uses half of it)
constexpr int kEpiBytes = kEpiWarps * kEpiBufBytes;  // one staging buffer per epilogue warp
constexpr int kRefBBytes = kTN * 4;                 // refB of the current tile
// CG = 1: one CTA per 128 x 256 tile, 4 stages of (A 128 x 128 + B 256 x 128) bytes.
// CG = 2: a pair of CTAs (cta_group::2) per 256 x 256 tile; each CTA stages its 128 rows of A and its 128-row half of
//         B, 6 stages of 32 KB: a third less shared-memory fill per MMA cycle, which is what bounds the main loop.
template <int CG> struct TcCfg {
    static constexpr int kBRows = CG == 2 ? 128 : 256;
    static constexpr int kBStage = kBRows * kTK;
    static constexpr int kStages = CG == 2 ? 6 : 4;
    static constexpr int kRing = kStages * (kAStage + kBStage);
};
static_assert(TcCfg<1>::kRing == TcCfg<2>::kRing, "both configurations use the same ring size");
constexpr int kMaxStages = 6;
// layout: operand ring | epilogue staging | refB | barriers.  The dynamic shared-memory base is 1024-byte aligned.
constexpr int kOffEpi = TcCfg<1>::kRing;
constexpr int kOffRefB = kOffEpi + kEpiBytes;
constexpr int kOffBars = kOffRefB + kRefBBytes;
constexpr int kTcSmem = kOffBars + kBarrierBytes;
constexpr int kTmemCols = 512;
constexpr int kDMax = 12, kDMin = -14;              // exponent window of a row, relative to its reference

// ------------------------------------------------------------------------------------------------------------------
// decode
// ------------------------------------------------------------------------------------------------------------------

struct DecodeOperand {
    const uint8_t *codes;
    const float *scales;
    int64_t ldc, lds, rows;
    int grid;
    uint8_t *out8;      // [rows][K]
    float *ref;         // [rows]
};

struct DecodeParams {
    DecodeOperand op[2];    // A and B in one launch
    int64_t K;
    int64_t a_ctas;         // CTAs [0, a_ctas) work on A, the next ones on B
    int64_t tbl_cta;        // this CTA (if launched) lists the row tiles of a row-grouped product
    const int64_t *offsets; // row offsets of the groups (device), num_groups + 1 of them
    int num_groups;
    int2 *mtiles;           // (first row, group) of every 256-row tile, group by group
    int32_t *dev_status;
};

constexpr int kDecodeThreads = 256;

// A CTA decodes 256 / TPR rows with TPR threads (32..256) on each: short rows keep a warp per row, long rows are
// spread over more threads so that the grid has many more warps than the GPU has slots (no idle tail).
template <int TPR, bool OWN>
__global__ void __launch_bounds__(kDecodeThreads) decode_rows_kernel(const DecodeParams P) {
    // the product kernel of the same call is launched as a programmatic dependent: its CTAs may take the SMs this grid's
    // last wave leaves free and set themselves up; they read nothing of this grid's output before griddepcontrol.wait
    asm volatile("griddepcontrol.launch_dependents;");
    constexpr int kRowsPerCta = kDecodeThreads / TPR;
    if ((int64_t)blockIdx.x == P.tbl_cta) {
        if (threadIdx.x == 0) {
            int n = 0;
            for (int g = 0; g < P.num_groups; ++g)
                for (int64_t m = P.offsets[g]; m < P.offsets[g + 1]; m += 2 * kTM) P.mtiles[n++] = make_int2((int)m, g);
        }
        return;
    }
    const bool is_b = (int64_t)blockIdx.x >= P.a_ctas;
    const DecodeOperand &O = P.op[is_b ? 1 : 0];
    const int lane = threadIdx.x & 31;
    const int t = threadIdx.x % TPR;
    const int64_t row = ((int64_t)blockIdx.x - (is_b ? P.a_ctas : 0)) * kRowsPerCta + threadIdx.x / TPR;
    const bool active = row < O.rows;
    const int nkb = (int)(P.K >> 4);
    const float *sptr = O.scales + (active ? row : 0) * O.lds + t;
    const uint2 *cptr = reinterpret_cast<const uint2 *>(O.codes + (active ? row : 0) * O.ldc) + t;

    // the thread's first kPre blocks (codes and exponent fields) are requested before the scan below, so that their
    // trip to DRAM overlaps the scan's
    constexpr int kPre = 4;
    uint2 pcw[kPre];
    int pf[kPre];
#pragma unroll
    for (int u = 0; u < kPre; ++u) {
        const bool in = active && t + u * TPR < nkb;
        pcw[u] = in ? __ldg(cptr + u * TPR) : make_uint2(0u, 0u);
        pf[u] = in ? (int)(__float_as_uint(__ldg(sptr + u * TPR)) >> 23) : 0;   // scales are non-negative: no sign bit
    }

    // largest block exponent field of the row (power-of-two scales: the exponent field is the scale; 0 = zero block),
    // eight loads in flight per thread.  OWN (a warp per row, or rows spread over four or eight warps): a thread scans
    // the scales of its own blocks only (the first of them are already in registers), the lanes of a warp combine by
    // shuffles and the warps of a row through shared memory.  Otherwise (two warps per row) both warps scan the whole
    // row (the repeats hit in cache) and no barrier is needed.
    int fmax = 0;
    if (OWN) {
#pragma unroll
        for (int u = 0; u < kPre; ++u) fmax = max(fmax, pf[u]);
        if (active) {
            int kb = t + kPre * TPR;
            for (; kb + 7 * TPR < nkb; kb += 8 * TPR) {
                uint32_t b[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) b[u] = __float_as_uint(__ldg(sptr + (kb - t) + u * TPR));
#pragma unroll
                for (int u = 0; u < 8; ++u) fmax = max(fmax, (int)(b[u] >> 23));
            }
            for (; kb < nkb; kb += TPR) fmax = max(fmax, (int)(__float_as_uint(__ldg(sptr + (kb - t))) >> 23));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) fmax = max(fmax, __shfl_xor_sync(0xFFFFFFFFu, fmax, o));
        if (TPR > 32) {
            __shared__ int wmax[kDecodeThreads / 32];
            if (lane == 0) wmax[threadIdx.x >> 5] = fmax;
            __syncthreads();
            const int w0 = (threadIdx.x / TPR) * (TPR / 32);
#pragma unroll
            for (int i = 0; i < TPR / 32; ++i) fmax = max(fmax, wmax[w0 + i]);
        }
    } else {
        uint32_t fm = 0u;
        if (active) {
            const float *srow0 = sptr - t;
            int kb = lane;
            for (; kb + 7 * 32 < nkb; kb += 8 * 32) {
                uint32_t b[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) b[u] = __float_as_uint(__ldg(srow0 + kb + u * 32));
#pragma unroll
                for (int u = 0; u < 8; ++u) fm = max(fm, b[u]);
            }
            for (; kb < nkb; kb += 32) fm = max(fm, __float_as_uint(__ldg(srow0 + kb)));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) fm = max(fm, __shfl_xor_sync(0xFFFFFFFFu, fm, o));
        fmax = (int)(fm >> 23);
    }
    if (!active) return;
    // biased exponent field of the row's reference 2^eref, eref = emax - kDMax (an all-zero row takes eref = 0)
    const int fref = fmax == 0 ? 127 : fmax - kDMax;
    if (t == 0) {
        // unit * 2^eref as two exact factors (fref may be below the smallest normal exponent field)
        const float unit = O.grid == UFP4_GRID_INT4 ? 1.0f : (O.grid == UFP4_GRID_E1M2 ? 0.25f : 0.5f);
        const int h = fref >= 1 ? fref : 1;
        O.ref[row] = __fmul_rn(__fmul_rn(unit, __uint_as_float((uint32_t)(127 + fref - h) << 23)), __uint_as_float((uint32_t)h << 23));
    }

    // E5M2 bytes of a grid's values at d = 0: magnitude 2^k (1 + f/4) -> (15 + k) << 2 | f, bit 7 = sign.  A nibble n
    // indexes a 16-entry table held in four registers: entries 0..7 (n < 8) and 8..15 (n >= 8, index n & 7).
    // Uniform grids: magnitudes 0..7 (INT4 two's complement: n >= 8 is n - 16, i.e. -8..-1; E1M2: sign | magnitude).
    // E2M1 (2 * value): 0, 1, 2, 3, 4, 6, 8, 12.  The negative zero of the sign | magnitude grids decodes to 0.
    const bool int4 = O.grid == UFP4_GRID_INT4;
    const uint32_t lutp_lo0 = 0x42403C00u;
    const uint32_t lutp_hi0 = O.grid == UFP4_GRID_E2M1 ? 0x4A484644u : 0x47464544u;
    const uint32_t lutn_lo0 = int4 ? 0xC5C6C7C8u : (lutp_lo0 | 0x80808000u);
    const uint32_t lutn_hi0 = int4 ? 0xBCC0C2C4u : (lutp_hi0 | 0x80808080u);
    const uint32_t mul_nlo = int4 ? 0x04040404u : 0x04040400u;     // a zero entry stays zero
    const int fkeep = max(1, fref + kDMin);                        // smallest exponent field that is not flushed
    uint32_t flushed = 0u;
    uint4 *optr = reinterpret_cast<uint4 *>(O.out8 + row * P.K) + t;
    auto emit = [&](int f, uint2 cw, uint4 *dst) {
        // a zero-scale or flushed block decodes as all-zero codes (table entry 0 is 0 at every d)
        const bool keep = f >= fkeep;
        flushed |= (keep || f == 0) ? 0u : (cw.x | cw.y);
        cw.x = keep ? cw.x : 0u;
        cw.y = keep ? cw.y : 0u;
        // per-block table: 4 d is added to each non-zero entry; the low 7 bits of every entry stay inside [4, 0x7A], so
        // the 32-bit wrap-around arithmetic below is an exact per-byte addition also for negative d
        const uint32_t d = (uint32_t)(f - fref);
        const uint32_t lutp_lo = lutp_lo0 + d * 0x04040400u, lutp_hi = lutp_hi0 + d * 0x04040404u;
        const uint32_t lutn_lo = lutn_lo0 + d * mul_nlo, lutn_hi = lutn_hi0 + d * 0x04040404u;
        uint32_t out[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            // four nibbles: look the low three bits up in both halves of the table, then take byte k from the half that
            // bit 3 of nibble k names (selector nibble k = k, or 4 + k)
            const uint32_t w = (q & 2 ? cw.y : cw.x) >> (q & 1 ? 16 : 0);
            const uint32_t sel = w & 0x7777u;
            const uint32_t pos = __byte_perm(lutp_lo, lutp_hi, sel), neg = __byte_perm(lutn_lo, lutn_hi, sel);
            out[q] = __byte_perm(pos, neg, ((w >> 1) & 0x4444u) | 0x3210u);
        }
        *dst = make_uint4(out[0], out[1], out[2], out[3]);
    };
#pragma unroll
    for (int u = 0; u < kPre; ++u)
        if (t + u * TPR < nkb) emit(pf[u], pcw[u], optr + u * TPR);
    cptr += kPre * TPR; optr += kPre * TPR; sptr += kPre * TPR;
#pragma unroll 4
    for (int kb = t + kPre * TPR; kb < nkb; kb += TPR, cptr += TPR, optr += TPR, sptr += TPR)
        emit((int)(__float_as_uint(__ldg(sptr)) >> 23), __ldg(cptr), optr);
    if (flushed != 0u && P.dev_status) atomicOr(P.dev_status, (int)UFP4_DEV_EXP_WINDOW);
}

// QMODE 0: C leaves as FP32 or BF16.  QMODE 1 / 2 (quantizing epilogue, plain products only): C is rounded to BF16 and
// quantized on the way out like ufp4_quantize would quantize it (uniform INT4 grid, RTNE, 1 x 16 blocks along N and
// along M, 16-point RHT or none; FP32 scales for QMODE 1, power-of-two scales for QMODE 2); the BF16 C itself is
// written only if P.C is given.
template <int CG, int QMODE = 0>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmC, const TcParams P) {
    using Cfg = TcCfg<CG>;
    constexpr int kStages = Cfg::kStages, kBStage = Cfg::kBStage;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = smem_u32(smem);
    const uint32_t sA = base, sB = base + kStages * kAStage;
    const uint32_t bars = base + kOffBars;
    const uint32_t full_bar = bars, empty_bar = bars + 8 * kMaxStages;
    const uint32_t tfull_bar = bars + 16 * kMaxStages, tempty_bar = tfull_bar + 16;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + kOffBars + 16 * kMaxStages + 32);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + kOffBars + 160);   // flag, poll limit
    const uint32_t rb_bar = bars + 16 * kMaxStages + 40;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // position in the group of CG CTAs that share an output tile; rank 0 issues the MMAs and owns the barriers the
    // pair synchronises on (operands landed, accumulator drained)
    const int rank = CG == 2 ? (int)cluster_cta_rank() : 0;
    const int group_id = blockIdx.x / CG, num_groups_launched = gridDim.x / CG;
    const uint32_t lead_full_bar = CG == 2 ? map_to_cta(full_bar, 0) : full_bar;
    const uint32_t lead_tempty_bar = CG == 2 ? map_to_cta(tempty_bar, 0) : tempty_bar;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar + 8 * s, CG);            // one arrive.expect_tx per CTA of the group
            mbar_init(empty_bar + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull_bar + 8 * a, 1);
            mbar_init(tempty_bar + 8 * a, CG * kEpiWarps);
            mbar_init(rb_bar + 8 * a, 32 * kEpiWarps);
        }
        abort_flag[0] = (base & 1023u) ? 1u : 0u;    // the swizzled layouts below need the 1024-byte alignment
        abort_flag[1] = P.wait_limit ? P.wait_limit : kWaitLimit;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        tmem_alloc<CG>(smem_u32((const void *)tmem_slot), kTmemCols);
    }
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();                   // the peer's barriers exist before anything is signalled on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // everything above is independent of the decode pass; its output (operand bytes, row references, tile list) is complete
    // and visible from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer: this CTA's 128 rows of A and its part of B
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = group_id; ok && !P.skip_loads && tile < P.total_tiles; tile += num_groups_launched) {
                const TileInfo t = tile_info<CG>(P, tile, rank);
                for (int kb = 0; kb < t.nkb; ++kb) {
                    if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const int32_t kc = (t.kb0 + kb) * kTK;
                    if (CG == 1) {
                        mbar_expect_tx(full_bar + 8 * stage, kAStage + kBStage);
                        tma_load_2d(sA + stage * kAStage, &tmA, kc, (int32_t)t.m0, full_bar + 8 * stage);
                        tma_load_2d(sB + stage * kBStage, &tmB, kc, (int32_t)(t.b_row0 + t.n0), full_bar + 8 * stage);
                    } else {
                        const uint32_t fb = lead_full_bar + 8 * stage;
                        if (rank == 0) mbar_expect_tx(full_bar + 8 * stage, kAStage + kBStage);
                        else mbar_expect_tx_cluster(fb, kAStage + kBStage);
                        tma_load_2d_pair(sA + stage * kAStage, &tmA, kc, (int32_t)t.m0, fb);
                        tma_load_2d_pair(sB + stage * kBStage, &tmB, kc, (int32_t)(t.b_row0 + t.n0 + rank * Cfg::kBRows), fb);
                    }
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // ---------------- MMA issuer (rank 0 of the group)
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = group_id; ok && tile < P.total_tiles; tile += num_groups_launched) {
                const TileInfo t = tile_info<CG>(P, tile, rank);
                if (t.nkb == 0) continue;
                if (!mbar_wait(tempty_bar + 8 * acc, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * kTN;
                for (int kb = 0; kb < t.nkb; ++kb) {
                    if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t adesc = umma_desc_sw128(sA + stage * kAStage);
                    const uint64_t bdesc = umma_desc_sw128(sB + stage * kBStage);
#pragma unroll
                    for (int k = 0; k < kTK / kUmmaK; ++k) {
                        // advancing K inside the 128-byte swizzle span: +32 bytes = +2 in the (address >> 4) field
                        tc_mma_f8<CG>(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), InstrDesc<CG>::value,
                                      (kb > 0 || k > 0) ? 1u : 0u);
                    }
                    tc_commit<CG>(empty_bar + 8 * stage);  // the stage is free (in every CTA of the group) once read
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit<CG>(tfull_bar + 8 * acc);        // accumulator complete (in every CTA of the group)
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1u;
            }
        }
    } else {
        // ---------------- epilogue: TMEM -> registers -> x refA[m] refB[n] -> swizzled shared staging -> TMA store of C
        // A thread owns one accumulator row; per 32-column chunk it writes its 128 (FP32) or 64 (BF16) bytes into the
        // warp's staging buffer in the 128B / 64B swizzle pattern and one lane hands the 32 x 32 box to the TMA, which
        // clips rows >= M and columns >= N.  Staging is double-buffered so the next chunk is prepared while the
        // previous box is still being read.
        const int q = warp & 3;                            // TMEM lane quarter this warp may access
        const int half = (warp - 2) >> 2;                  // which four of the eight 32-column chunks this warp drains
        const int et = threadIdx.x - 64;                   // 0..255 among the epilogue threads
        uint8_t *buf = smem + kOffEpi + (warp - 2) * kEpiBufBytes;
        float *refb_s = reinterpret_cast<float *>(smem + kOffRefB);
        int acc = 0;
        uint32_t acc_phase = 0, rb_written = 0, rb_read = 0;
        bool first_tile = true;
        bool ok = true;
        for (int tile = group_id; ok && tile < P.total_tiles; tile += num_groups_launched) {
            const TileInfo t = tile_info<CG>(P, tile, rank);
            const int64_t m_own = t.m0 + q * 32 + lane;
            const float ra = m_own < P.M ? P.refA[m_own] : 0.0f;
            // refB of this tile's 256 columns into shared memory (one value per thread)
            {
                const int64_t n = t.n0 + et;
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
            if (t.nkb > 0) {
                if (!mbar_wait_warp(tfull_bar + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
                tc_fence_after();
            }
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)acc * kTN;
            const int32_t c_row = (int32_t)(t.m0 + q * 32), c_grp = (int32_t)(t.c_row0 / (P.M > 0 ? P.M : 1));
            uint32_t v[2][32];
            const int c_begin = 4 * half;
            if (t.nkb > 0) tc_ld32(taddr + (uint32_t)(c_begin * 32), v[0]);
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const int c = c_begin + cc, cur = cc & 1;
                if (t.nkb > 0) {
                    tc_wait_ld();
                    if (cc + 1 < 4) tc_ld32(taddr + (uint32_t)((c + 1) * 32), v[cur ^ 1]);
                    else {
                        // every column of this accumulator has been read: hand it back to the MMA warp
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) {
                            if (CG == 1) mbar_arrive(tempty_bar + 8 * acc);
                            else mbar_arrive_cluster(lead_tempty_bar + 8 * acc);
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[cur][j] = 0u;
                }
                const int64_t n_base = t.n0 + c * 32;
                if (n_base >= P.N || c_row >= t.row_end) continue;     // warp-uniform: the whole box is clipped or not this tile's
                if (n_base + 32 > P.N && P.n_unaligned) {
                    float x[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) x[j] = __uint_as_float(v[cur][j]) * ra * refb_s[c * 32 + j];
                    epi_store_box_plain(P, x, t.c_row0 + m_own, n_base, m_own < t.row_end);
                    continue;
                }
                if (QMODE != 0) {
                    // the previous box must have been read out of the staging buffer by its TMA store
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    __syncwarp();
                    // ---- quantizing epilogue.  The BF16-rounded 32 x 32 box goes to the staging buffer in the BF16 store's
                    // layout (64-byte rows, 16-byte piece j of row r at piece j ^ ((r >> 1) & 3)); the words a thread
                    // builds for it, two adjacent columns each, are what the quantizer's row pass starts from.
                    constexpr int QF = QMODE == 1 ? UFP4_SCALE_FP32 : UFP4_SCALE_POW2;
                    uint32_t w[16];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float4 r0 = rb4[c * 8 + 2 * j], r1 = rb4[c * 8 + 2 * j + 1];
                        const uint32_t *x = &v[cur][8 * j];
                        __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(x[0]) * ra * r0.x, __uint_as_float(x[1]) * ra * r0.y);
                        __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(x[2]) * ra * r0.z, __uint_as_float(x[3]) * ra * r0.w);
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(x[4]) * ra * r1.x, __uint_as_float(x[5]) * ra * r1.y);
                        __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(x[6]) * ra * r1.z, __uint_as_float(x[7]) * ra * r1.w);
                        w[4 * j] = *reinterpret_cast<uint32_t *>(&h0); w[4 * j + 1] = *reinterpret_cast<uint32_t *>(&h1);
                        w[4 * j + 2] = *reinterpret_cast<uint32_t *>(&h2); w[4 * j + 3] = *reinterpret_cast<uint32_t *>(&h3);
                        *reinterpret_cast<uint4 *>(buf + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)) =
                            make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                    }
                    const QuantParams QP = {};                          // not read on the uniform-grid RTNE path
                    bool nonfinite = false;
                    if (P.q_row_codes) {
                        // blocks along N: columns n_base .. +15 (words 0..7) and +16 .. +31 (words 8..15) of this thread's row
                        float2 qv[16];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const uint32_t sl = P.q_rht ? P.q_sign_lo[j] : 0u, sh = P.q_rht ? P.q_sign_hi[j] : 0u;
                            qv[2 * j] = make_float2(__uint_as_float(w[j] * 65536u + sl), __uint_as_float(w[8 + j] * 65536u + sl));
                            qv[2 * j + 1] = make_float2(__uint_as_float((w[j] & 0xFFFF0000u) ^ sh), __uint_as_float((w[8 + j] & 0xFFFF0000u) ^ sh));
                        }
                        uint2 c0, c1;
                        uint32_t s0, s1;
                        if (P.q_rht) quantize_pair<GC_INT4, UFP4_ROUND_RTNE, QF, true>(qv, QP, 1.0f, 0, 0, 0u, &c0, &c1, &s0, &s1, &nonfinite);
                        else quantize_pair<GC_INT4, UFP4_ROUND_RTNE, QF, false>(qv, QP, 1.0f, 0, 0, 0u, &c0, &c1, &s0, &s1, &nonfinite);
                        if (m_own < t.row_end) {
                            uint8_t *dst = P.q_row_codes + m_own * P.q_row_ldc + (n_base >> 1);
                            float *sd = P.q_row_scales + m_own * P.q_row_lds + (n_base >> 4);
                            if (n_base + 32 <= P.N) {
                                *reinterpret_cast<uint4 *>(dst) = make_uint4(c0.x, c0.y, c1.x, c1.y);
                                reinterpret_cast<uint32_t *>(sd)[0] = s0;
                                reinterpret_cast<uint32_t *>(sd)[1] = s1;
                            } else {                                   // N is a multiple of 16: the first block is inside
                                *reinterpret_cast<uint2 *>(dst) = c0;
                                *reinterpret_cast<uint32_t *>(sd) = s0;
                            }
                        }
                    }
                    __syncwarp();
                    if (P.q_col_codes) {
                        // blocks along M: lane j takes column n_base + j of the staged box, rows 0..15 and 16..31
                        const int64_t n_own = n_base + lane;
                        float2 qv[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const uint32_t sc = P.q_rht ? P.q_sign[i] : 0u;
                            const int r0i = i, r1i = 16 + i;
                            const uint32_t e0 = *reinterpret_cast<const uint16_t *>(buf + r0i * 64 + (((lane >> 3) ^ ((r0i >> 1) & 3)) << 4) + ((lane & 7) << 1));
                            const uint32_t e1 = *reinterpret_cast<const uint16_t *>(buf + r1i * 64 + (((lane >> 3) ^ ((r1i >> 1) & 3)) << 4) + ((lane & 7) << 1));
                            qv[i] = make_float2(__uint_as_float(e0 * 65536u + sc), __uint_as_float(e1 * 65536u + sc));
                        }
                        uint2 c0, c1;
                        uint32_t s0, s1;
                        if (P.q_rht) quantize_pair<GC_INT4, UFP4_ROUND_RTNE, QF, true>(qv, QP, 1.0f, 0, 0, 0u, &c0, &c1, &s0, &s1, &nonfinite);
                        else quantize_pair<GC_INT4, UFP4_ROUND_RTNE, QF, false>(qv, QP, 1.0f, 0, 0, 0u, &c0, &c1, &s0, &s1, &nonfinite);
                        if (n_own < P.N) {
                            uint8_t *dst = P.q_col_codes + n_own * P.q_col_ldc + (c_row >> 1);
                            float *sd = P.q_col_scales + n_own * P.q_col_lds + (c_row >> 4);
                            if (c_row + 32 <= t.row_end) {
                                *reinterpret_cast<uint4 *>(dst) = make_uint4(c0.x, c0.y, c1.x, c1.y);
                                reinterpret_cast<uint32_t *>(sd)[0] = s0;
                                reinterpret_cast<uint32_t *>(sd)[1] = s1;
                            } else {                                   // M is a multiple of 16: the first block is inside
                                *reinterpret_cast<uint2 *>(dst) = c0;
                                *reinterpret_cast<uint32_t *>(sd) = s0;
                            }
                        }
                    }
                    if (nonfinite && P.dev_status) atomicOr(P.dev_status, (int)UFP4_DEV_NONFINITE);
                    if (!P.C) {                                        // no BF16 copy of C wanted: nothing for the TMA to store
                        __syncwarp();
                        continue;
                    }
                } else {
                    float x[32];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float4 r = rb4[c * 8 + j];
                        x[4 * j] = __uint_as_float(v[cur][4 * j]) * ra * r.x;
                        x[4 * j + 1] = __uint_as_float(v[cur][4 * j + 1]) * ra * r.y;
                        x[4 * j + 2] = __uint_as_float(v[cur][4 * j + 2]) * ra * r.z;
                        x[4 * j + 3] = __uint_as_float(v[cur][4 * j + 3]) * ra * r.w;
                    }
                    epi_store_box_tma(P, &tmC, buf, lane, x, (int32_t)n_base, c_row, c_grp);
                    continue;
                }
                // QMODE with a BF16 copy of C: the box is already staged
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) {
                    asm volatile(
                        "cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                        ::"l"(&tmC), "r"((int32_t)n_base), "r"(c_row), "r"(c_grp), "r"(smem_u32(buf)) : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                }
            }
            mbar_arrive(rb_bar + 8);                           // this thread has finished with the tile's refB values
            if (t.nkb > 0) {
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1u;
            }
        }
        epi_store_drain(lane);
    }
    tc_teardown<CG>(abort_flag, P.dev_status, tmem_base, kTmemCols, warp);
}

// ------------------------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------------------------

static bool make_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t K, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K};
    cuuint32_t box[2] = {(cuuint32_t)kTK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// decoded operands, reference vectors, and the row-tile list of a row-grouped product (at most one tile per 128 rows)
size_t gemm_tensor_workspace_bytes(int64_t a_rows, int64_t b_rows, int64_t K) {
    return round_up((size_t)a_rows * K, 256) + round_up((size_t)b_rows * K, 256) + round_up((size_t)a_rows * 4, 256) +
           round_up((size_t)b_rows * 4, 256) + round_up((size_t)(a_rows / 128 + 2) * sizeof(int2), 256);
}

int gemm_tensor_kernel_launches() { return 2; }

bool gemm_tensor_supported(const ufp4_qtensor *A, const ufp4_qtensor *B, int64_t M, int64_t N, int64_t K, int mode) {
    (void)mode;
    if (!is_pow2_fmt(A->scale_fmt) || !is_pow2_fmt(B->scale_fmt)) return false;
    if (K % 16 != 0 || M < 1 || N < 1) return false;
    if (A->rows > 0x7FFFFFFF || B->rows > 0x7FFFFFFF || K > 0x7FFFFFFF) return false;
    return true;
}

// qout (optional): the quantizing epilogue's outputs and settings; then C is BF16 or NULL and mode is 0.
int gemm_tensor_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int mode,
                       int64_t M, int64_t N, int64_t K, const int64_t *offsets, const int64_t *host_offsets,
                       int num_groups, int64_t group_n, void *workspace, size_t workspace_bytes, int32_t *dev_status,
                       void *stream, const TcQOut *qout) {
    if (!aligned_to(workspace, 256)) return UFP4_ERR_ALIGN;
    if (workspace_bytes < gemm_tensor_workspace_bytes(A->rows, B->rows, K)) return UFP4_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    uint8_t *A8 = ws;
    uint8_t *B8 = A8 + round_up((size_t)A->rows * K, 256);
    float *refA = reinterpret_cast<float *>(B8 + round_up((size_t)B->rows * K, 256));
    float *refB = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(refA) + round_up((size_t)A->rows * 4, 256));
    int2 *mtiles = reinterpret_cast<int2 *>(reinterpret_cast<uint8_t *>(refB) + round_up((size_t)B->rows * 4, 256));
    // CTA pairs (cta_group::2), except for row-grouped products with a short reduction: those are bound by writing C, and
    // single CTAs on 128-row tiles waste nothing on groups of 128 (mod 256) rows
    const int cg = (mode == 1 && K < 4096) ? 1 : 2;
    // row-grouped product on pairs: 256-row tiles group by group (the decode launch lists them from the device offsets)
    int64_t row_tiles = 0;
    if (mode == 1) {
        if (A->rows > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
        for (int g = 0; g < num_groups; ++g) row_tiles += (host_offsets[g + 1] - host_offsets[g] + 2 * kTM - 1) / (2 * kTM);
    }

    DecodeParams D = {};
    D.op[0] = DecodeOperand{static_cast<const uint8_t *>(A->codes), static_cast<const float *>(A->scales),
                            A->ld_codes_bytes, A->ld_scales, A->rows, codebook_of(A->grid), A8, refA};
    D.op[1] = DecodeOperand{static_cast<const uint8_t *>(B->codes), static_cast<const float *>(B->scales),
                            B->ld_codes_bytes, B->ld_scales, B->rows, codebook_of(B->grid), B8, refB};
    D.K = K;
    int tpr = 32;           // a warp per row up to 8 blocks per thread, more threads on longer rows
    while (tpr < kDecodeThreads && (K >> 4) >= (int64_t)16 * tpr) tpr *= 2;
    const int64_t rows_per_cta = kDecodeThreads / tpr;
    D.a_ctas = (A->rows + rows_per_cta - 1) / rows_per_cta;
    D.dev_status = dev_status;
    D.tbl_cta = D.a_ctas + (B->rows + rows_per_cta - 1) / rows_per_cta;
    D.offsets = offsets; D.num_groups = num_groups; D.mtiles = mtiles;
    const int64_t decode_ctas = D.tbl_cta + (mode == 1 && cg == 2 ? 1 : 0);
    if (decode_ctas > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    const unsigned dg = (unsigned)decode_ctas;
    // a warp per row, or rows spread over four or eight warps: each thread scans only its own blocks' scales (the warps of
    // a row combine through shared memory); with two warps per row both scan the whole row (no barrier; measured faster)
    if (tpr == 32) decode_rows_kernel<32, true><<<dg, kDecodeThreads, 0, st>>>(D);
    else if (tpr == 64) decode_rows_kernel<64, false><<<dg, kDecodeThreads, 0, st>>>(D);
    else if (tpr == 128) decode_rows_kernel<128, true><<<dg, kDecodeThreads, 0, st>>>(D);
    else decode_rows_kernel<256, true><<<dg, kDecodeThreads, 0, st>>>(D);
    if (cudaGetLastError() != cudaSuccess) return UFP4_ERR_CUDA;

    CUtensorMap tmA, tmB;
    if (!make_map(&tmA, A8, A->rows, K, kTM) || !make_map(&tmB, B8, B->rows, K, cg == 2 ? TcCfg<2>::kBRows : TcCfg<1>::kBRows))
        return UFP4_ERR_CUDA;

    // C as [groups][rows][cols] so that the TMA store clips at the end of each group's rows and at N
    CUtensorMap tmC = {};
    if (C) {
        EncodeTiledFn fn = encode_tiled_fn();
        if (!fn) return UFP4_ERR_CUDA;
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
    P.mt = (mode == 1 && cg == 2) ? (int)row_tiles : (int)((M + kTM * cg - 1) / (kTM * cg));
    P.nt = (int)((N + kTN - 1) / kTN);
    const int64_t total = (int64_t)P.mt * P.nt * (mode == 2 ? num_groups : 1);
    if (total < 1 || total > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    P.total_tiles = (int)total;
    P.n_unaligned = ((N * (c_is_bf16 ? 2 : 4)) % 16) != 0;
    P.wait_limit = debug_wait_limit();
    P.skip_loads = debug_skip_loads();
    int qmode = 0;
    if (qout) {
        qmode = qout->pow2 ? 2 : 1;
        P.q_row_codes = qout->row_codes; P.q_row_scales = qout->row_scales; P.q_row_ldc = qout->row_ldc; P.q_row_lds = qout->row_lds;
        P.q_col_codes = qout->col_codes; P.q_col_scales = qout->col_scales; P.q_col_ldc = qout->col_ldc; P.q_col_lds = qout->col_lds;
        P.q_rht = qout->rht;
        for (int j = 0; j < 8; ++j) {
            P.q_sign_lo[j] = ((qout->sign_mask >> (2 * j)) & 1u) << 31;
            P.q_sign_hi[j] = ((qout->sign_mask >> (2 * j + 1)) & 1u) << 31;
        }
        for (int i = 0; i < 16; ++i) P.q_sign[i] = ((qout->sign_mask >> i) & 1u) << 31;
    }

    static DeviceSetup slots[kMaxDevices];
    const DeviceSetup *dev = nullptr;
    const int rc_setup = device_setup(slots, [](int ordinal, DeviceSetup &d) -> int {
        UFP4_CUDA_OK(cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, ordinal));
        UFP4_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem));
        UFP4_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem));
        UFP4_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel<2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem));
        UFP4_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem));
        d.max_pairs = resident_pairs(gemm_tc_kernel<2>, kTcThreads, kTcSmem, d.num_sms);
        if (getenv("UFP4_DEBUG")) fprintf(stderr, "[ufp4] device %d: SMs %d, resident CTA pairs %d\n", ordinal, d.num_sms, d.max_pairs);
        return UFP4_OK;
    }, &dev);
    if (rc_setup != UFP4_OK) return rc_setup;
    const int num_sms = dev->num_sms, max_pairs = dev->max_pairs;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // dependent of the decode launch above
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = kTcSmem;
    cfg.stream = st;
    cfg.attrs = attr;
    if (cg == 1) {
        cfg.gridDim = dim3((unsigned)(total < num_sms ? total : num_sms));
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<1>, tmA, tmB, tmC, P) == cudaSuccess ? UFP4_OK : UFP4_ERR_CUDA;
    }
    cfg.gridDim = dim3(2 * (unsigned)(total < max_pairs ? total : max_pairs));
    cfg.numAttrs = 2;
    cudaError_t err;
    if (qmode == 1) err = cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2, 1>, tmA, tmB, tmC, P);
    else if (qmode == 2) err = cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2, 2>, tmA, tmB, tmC, P);
    else err = cudaLaunchKernelEx(&cfg, gemm_tc_kernel<2>, tmA, tmB, tmC, P);
    return err == cudaSuccess ? UFP4_OK : UFP4_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------------------------
// Allocation-free variant of the tensor-core GEMM: its scratch lives in this file-scope device array, which every GPU
// that loads the library holds until the process exits.
// ------------------------------------------------------------------------------------------------------------------

constexpr size_t kNoAllocScratchBytes = (size_t)16 << 20;
static __device__ __align__(256) uint8_t g_noalloc_scratch[kNoAllocScratchBytes];

static std::atomic<void *> g_noalloc_ptr[kMaxDevices];

// Device address of the scratch array on the current device.  In host code the array's name is only a handle, not an
// address a kernel could use, so the address is asked for once per device (with that device current) and cached.
static int noalloc_scratch(void **out) {
    int dev = 0;
    UFP4_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return UFP4_ERR_UNSUPPORTED;
    void *p = g_noalloc_ptr[dev].load(std::memory_order_acquire);
    if (!p) {
        UFP4_CUDA_OK(cudaGetSymbolAddress(&p, g_noalloc_scratch));     // the same answer from every thread
        g_noalloc_ptr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return UFP4_OK;
}

int gemm_noalloc_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16,
                        int32_t *dev_status, void *stream) {
    if (!gemm_tensor_supported(A, B, A->rows, B->rows, A->k, 0)) return UFP4_ERR_UNSUPPORTED;
    if (gemm_tensor_workspace_bytes(A->rows, B->rows, A->k) > kNoAllocScratchBytes) return UFP4_ERR_WORKSPACE;
    void *scratch = nullptr;
    int rc = noalloc_scratch(&scratch);
    if (rc != UFP4_OK) return rc;
    return gemm_tensor_launch(A, B, C, ldc, c_is_bf16, 0, A->rows, B->rows, A->k, nullptr, nullptr, 1, B->rows, scratch,
                              kNoAllocScratchBytes, dev_status, stream, nullptr);
}

size_t gemm_noalloc_max_bytes() { return kNoAllocScratchBytes; }

}  // namespace ufp4
