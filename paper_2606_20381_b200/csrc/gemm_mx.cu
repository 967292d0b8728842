// Tensor-core path with HARDWARE block scaling (Sec. 2.1's footnote on MXFP4: 1 x 32 blocks with an E8M0 scale; Sec. 2.2:
// Y^ = Q_G(XH') Q_G(WH')^T) for power-of-two block scales: tcgen05.mma kind::mxf8f6f4 with one UE8M0 scale per 32
// elements of K and operand row, applied by the tensor core itself.
//
// The operand element is the bare code as an E5M2 byte (|q| <= 7 has three significant bits), times 2^(e - e32) where e
// is its 16-block's exponent and e32 the larger exponent of the two 16-blocks that share a hardware scale: zero for
// UFP4_SCALE_E8M0_B32 tensors (both halves carry the same scale), and a gap inside one 32-element group for
// UFP4_SCALE_POW2 tensors.  No per-row reference exponent, no row scan, and no window relative to the rest of the row:
// a block is flushed (and UFP4_DEV_EXP_WINDOW set) only if it lies more than 2^14 below the other half of its own
// 32-group, which a 1 x 32 tensor cannot do by construction.  Two kernels:
//   1. decode_mx_kernel: packed nibbles + scales -> E5M2 bytes [rows][K] and UE8M0 scale bytes in the 512-byte units the
//      tensor core's scale copy takes: unit (K step of 128, row tile of 128) holds byte (row r, 32-group j) at
//      (r % 32) * 16 + (r / 32) * 4 + j; units are stored [K step][row tile], so the two units of a 256-row B tile are
//      adjacent.
//   2. gemm_mx_kernel: persistent, warp-specialised, one CTA pair (cta_group::2) per 256 x 256 tile.  Each CTA's TMA
//      producer brings its 128 rows of A, its 128-row half of B, the scale unit of its A rows and both scale units of
//      the B tile into a 5-stage ring; the leader's MMA thread copies a stage's scales to tensor memory
//      (tcgen05.cp.cta_group::2 32x128b.warpx4: each CTA's own shared memory to its own tensor memory, 4 columns for A,
//      8 for B) and issues four block-scaled MMAs (M256 x N256 x K32, scale ids 0..3) into the FP32 accumulator; the
//      epilogue is the folded kernel's (tcgen05.ld, staging, TMA store).  Twelve scale columns beside a 256-column
//      accumulator leave no room for a second accumulator in the 512 columns, so the epilogue warps first drain the
//      whole accumulator into registers, hand it back, and only then convert and store: the next tile's main loop waits
//      for the drain, not for the stores.
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdlib.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tc.cuh"

namespace ufp4 {

constexpr int kMxStages = 5;
constexpr int kMxA = kTM * kTK;                       // 16 KB: this CTA's 128 rows of the pair's A tile
constexpr int kMxB = (kTN / 2) * kTK;                 // 16 KB: this CTA's 128-row half of the B tile
constexpr int kMxSfUnit = 512;                        // scales of 128 rows x 4 groups of 32
constexpr int kMxSfA = kMxSfUnit, kMxSfB = 2 * kMxSfUnit;         // own rows of A; all 256 rows of the B tile
constexpr int kMxStageBytes = kMxA + kMxB + kMxSfA + kMxSfB;      // what one CTA's producer brings per stage
constexpr int kMxEpiWarps = 8;
constexpr int kMxThreads = 64 + 32 * kMxEpiWarps;
// layout: [A tiles][B tiles][scale units][epilogue staging][barriers]; operand tiles and staging 1024-byte aligned
constexpr int kMxOffB = kMxStages * kMxA;
constexpr int kMxOffSf = kMxOffB + kMxStages * kMxB;
constexpr int kMxOffEpi = (kMxOffSf + kMxStages * (kMxSfA + kMxSfB) + 1023) / 1024 * 1024;    // swizzled staging boxes
constexpr int kMxOffBars = kMxOffEpi + kMxEpiWarps * 4096;
constexpr int kMxSmem = kMxOffBars + 256;
static_assert(kMxOffEpi % 1024 == 0 && kMxOffB % 1024 == 0 && kMxOffSf % 128 == 0 && kMxSmem <= 227 * 1024, "shared-memory layout");
static_assert(16 * kMxStages + 24 <= 160, "barriers, the tensor-memory slot and the abort flag share 256 bytes");
constexpr int kMxDMin = -14;                          // smallest exponent gap an E5M2 element still holds exactly

// ------------------------------------------------------------------------------------------------------------------
// decode
// ------------------------------------------------------------------------------------------------------------------

struct MxOperand {
    const uint8_t *codes;
    const float *scales;
    int64_t ldc, lds, rows, rows_padded;   // rows_padded: multiple of 256 (whole scale units for every tile)
    int grid;
    uint8_t *out8;      // [rows][K]
    uint8_t *sf;        // [ksteps][rows_padded / 128][512]
};

struct MxDecodeParams {
    MxOperand op[2];
    int64_t K, ksteps;      // ksteps = ceil(K / 128)
    int64_t a_ctas;
    int32_t *dev_status;
};

// One thread per (row, 32-group): 8 threads cover a K step, 32 threads a 512-element stretch of a row.
__global__ void __launch_bounds__(256) decode_mx_kernel(const MxDecodeParams P) {
    // the product kernel of the same call is a programmatic dependent launch: see its griddepcontrol.wait
    asm volatile("griddepcontrol.launch_dependents;");
    const bool is_b = (int64_t)blockIdx.x >= P.a_ctas;
    const MxOperand &O = P.op[is_b ? 1 : 0];
    const int64_t ngroups = P.ksteps * 4;                                  // 32-groups per row, K padded to 128
    const int64_t gid = ((int64_t)blockIdx.x - (is_b ? P.a_ctas : 0)) * 256 + threadIdx.x;
    const int64_t row = gid / ngroups, g = gid - row * ngroups;
    if (row >= O.rows_padded) return;
    uint8_t *sf = O.sf + ((g >> 2) * (O.rows_padded >> 7) + (row >> 7)) * kMxSfUnit + ((row & 31) << 4) + (((row >> 5) & 3) << 2) + (g & 3);
    const int64_t nkb = P.K >> 4;
    if (row >= O.rows || 2 * g >= nkb) {
        *sf = 127;                           // padding: scale 1 on all-zero elements (the TMA fills them with zeros)
        return;
    }
    const bool has2 = 2 * g + 1 < nkb;       // K is a multiple of 16, not necessarily of 32
    const float *sp = O.scales + row * O.lds + 2 * g;
    const uint2 *cp = reinterpret_cast<const uint2 *>(O.codes + row * O.ldc) + 2 * g;
    const int f0 = (int)(__float_as_uint(__ldg(sp)) >> 23);                // power-of-two scales: the exponent field is the scale
    const int f1 = has2 ? (int)(__float_as_uint(__ldg(sp + 1)) >> 23) : 0;
    const uint2 c0 = __ldg(cp), c1 = has2 ? __ldg(cp + 1) : make_uint2(0u, 0u);
    const int fmax = max(f0, f1);
    *sf = (uint8_t)(fmax == 0 ? 127 : fmax);                               // UE8M0 has the FP32 exponent bias

    // E5M2 bytes of a grid's values: magnitude 2^k (1 + f/4) -> (15 + k) << 2 | f, bit 7 = sign; a nibble indexes a
    // 16-entry table held in four registers (see decode_rows_kernel); 4 d is added to every non-zero entry.
    const bool int4 = O.grid == UFP4_GRID_INT4;
    const uint32_t lutp_lo0 = 0x42403C00u;
    const uint32_t lutp_hi0 = O.grid == UFP4_GRID_E2M1 ? 0x4A484644u : 0x47464544u;
    const uint32_t lutn_lo0 = int4 ? 0xC5C6C7C8u : (lutp_lo0 | 0x80808000u);
    const uint32_t lutn_hi0 = int4 ? 0xBCC0C2C4u : (lutp_hi0 | 0x80808080u);
    const uint32_t mul_nlo = int4 ? 0x04040404u : 0x04040400u;
    uint32_t flushed = 0u;
    uint4 *optr = reinterpret_cast<uint4 *>(O.out8 + row * P.K) + 2 * g;
    auto emit = [&](int f, uint2 cw, uint4 *dst) {
        const bool keep = f != 0 && f - fmax >= kMxDMin;
        flushed |= (keep || f == 0) ? 0u : (cw.x | cw.y);
        cw.x = keep ? cw.x : 0u;
        cw.y = keep ? cw.y : 0u;
        const uint32_t d = keep ? (uint32_t)(f - fmax) : 0u;
        const uint32_t lutp_lo = lutp_lo0 + d * 0x04040400u, lutp_hi = lutp_hi0 + d * 0x04040404u;
        const uint32_t lutn_lo = lutn_lo0 + d * mul_nlo, lutn_hi = lutn_hi0 + d * 0x04040404u;
        uint32_t out[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint32_t w = (q & 2 ? cw.y : cw.x) >> (q & 1 ? 16 : 0);
            const uint32_t sel = w & 0x7777u;
            const uint32_t pos = __byte_perm(lutp_lo, lutp_hi, sel), neg = __byte_perm(lutn_lo, lutn_hi, sel);
            out[q] = __byte_perm(pos, neg, ((w >> 1) & 0x4444u) | 0x3210u);
        }
        *dst = make_uint4(out[0], out[1], out[2], out[3]);
    };
    emit(f0, c0, optr);
    if (has2) emit(f1, c1, optr + 1);
    if (flushed != 0u && P.dev_status) atomicOr(P.dev_status, (int)UFP4_DEV_EXP_WINDOW);
}

// ------------------------------------------------------------------------------------------------------------------
// product
// ------------------------------------------------------------------------------------------------------------------

// Shared-memory descriptor of a 512-byte scale unit for tcgen05.cp: 32 rows of 16 bytes, no swizzle, 8-row groups 128
// bytes apart.
__device__ __forceinline__ uint64_t sf_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)1u << 16;
    d |= (uint64_t)(128u >> 4) << 32;
    d |= (uint64_t)1u << 46;
    return d;
}
// One scale unit from shared to tensor memory, in both CTAs of the pair: each CTA copies from its own shared memory (same
// offset) into its own tensor memory (same column); 4 columns, the 128 bytes of a 32-row group replicated to the four
// lane quarters.
__device__ __forceinline__ void tc_cp_sf(uint32_t taddr, uint64_t desc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
// kind::mxf8f6f4, block-scaled, on a CTA pair: A = B = E5M2 (format 1), UE8M0 scales, both K-major, M = 256, N = 256;
// sf_id picks the byte (the 32-group of the K step) of the scale columns.
__device__ __forceinline__ void tc_mma_mx(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t sf_id, uint32_t t_sfa,
                                          uint32_t t_sfb, uint32_t accumulate) {
    const uint32_t idesc = (sf_id << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTN >> 3) << 17) | (1u << 23) |
                           ((uint32_t)((2 * kTM) >> 4) << 24) | (sf_id << 29);
    asm volatile(
        "{ .reg .pred p; setp.ne.b32 p, %6, 0; "
        "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale.scale_vec::1X [%0], %1, %2, %3, [%4], [%5], p; }"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(t_sfa), "r"(t_sfb), "r"(accumulate) : "memory");
}

struct MxArgs {
    int64_t a_tiles, b_tiles;    // 128-row tiles of the (padded) scale arrays: unit of (K step ks, tile t) is row ks * tiles + t
    float unit;                  // product of the two grids' code units
};

__global__ void __launch_bounds__(kMxThreads, 1)
gemm_mx_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmSfA, const __grid_constant__ CUtensorMap tmSfB,
               const __grid_constant__ CUtensorMap tmC, const TcParams P, const MxArgs X) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = smem_u32(smem);
    const uint32_t sA = base, sB = base + kMxOffB, sSf = base + kMxOffSf;
    const uint32_t bars = base + kMxOffBars;
    const uint32_t full_bar = bars, empty_bar = bars + 8 * kMxStages, tfull_bar = bars + 16 * kMxStages, tempty_bar = tfull_bar + 8;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + kMxOffBars + 16 * kMxStages + 16);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + kMxOffBars + 160);   // flag, poll limit
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // rank 0 of the pair issues the MMAs and owns the barriers the pair synchronises on
    const int rank = (int)cluster_cta_rank();
    const int group_id = blockIdx.x / 2, num_groups_launched = gridDim.x / 2;
    const uint32_t lead_full_bar = map_to_cta(full_bar, 0), lead_tempty_bar = map_to_cta(tempty_bar, 0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMxStages; ++s) {
            mbar_init(full_bar + 8 * s, 2);              // one arrive.expect_tx per CTA of the pair
            mbar_init(empty_bar + 8 * s, 1);
        }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, 2 * kMxEpiWarps);
        abort_flag[0] = (base & 1023u) ? 1u : 0u;
        abort_flag[1] = P.wait_limit ? P.wait_limit : kWaitLimit;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        tmem_alloc<2>(smem_u32((const void *)tmem_slot), 512);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                  // the peer's barriers exist before anything is signalled on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // the set-up above overlapped the decode pass's last wave; its output is complete and visible from here on
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t t_sfa = tmem_base + kTN, t_sfb = tmem_base + kTN + 4;     // accumulator: columns 0..255, then the scales

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer: this CTA's rows of A and of B, the scales of its A rows and of the whole B tile
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = group_id; ok && !P.skip_loads && tile < P.total_tiles; tile += num_groups_launched) {
                const TileInfo t = tile_info<2>(P, tile, rank);
                const int32_t ta = (int32_t)(t.m0 >> 7), tb = (int32_t)(t.n0 >> 7);
                for (int kb = 0; kb < t.nkb; ++kb) {
                    if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const int32_t ks = t.kb0 + kb;
                    const uint32_t fb = lead_full_bar + 8 * stage, sf = sSf + stage * (kMxSfA + kMxSfB);
                    if (rank == 0) mbar_expect_tx(full_bar + 8 * stage, kMxStageBytes);
                    else mbar_expect_tx_cluster(fb, kMxStageBytes);
                    tma_load_2d_pair(sA + stage * kMxA, &tmA, ks * kTK, (int32_t)t.m0, fb);
                    tma_load_2d_pair(sB + stage * kMxB, &tmB, ks * kTK, (int32_t)(t.n0 + rank * (kTN / 2)), fb);
                    tma_load_2d_pair(sf, &tmSfA, 0, (int32_t)(ks * X.a_tiles) + ta, fb);
                    tma_load_2d_pair(sf + kMxSfUnit, &tmSfB, 0, (int32_t)(ks * X.b_tiles) + tb, fb);
                    if (++stage == kMxStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // ---------------- MMA issuer (rank 0 of the pair)
            int stage = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = group_id; ok && tile < P.total_tiles; tile += num_groups_launched) {
                const TileInfo t = tile_info<2>(P, tile, rank);
                if (t.nkb == 0) continue;
                if (!mbar_wait(tempty_bar, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                for (int kb = 0; kb < t.nkb; ++kb) {
                    if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sf = sSf + stage * (kMxSfA + kMxSfB);
                    tc_cp_sf(t_sfa, sf_desc(sf));
                    tc_cp_sf(t_sfb, sf_desc(sf + kMxSfUnit));
                    tc_cp_sf(t_sfb + 4, sf_desc(sf + 2 * kMxSfUnit));
                    const uint64_t adesc = umma_desc_sw128(sA + stage * kMxA), bdesc = umma_desc_sw128(sB + stage * kMxB);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        tc_mma_mx(tmem_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), (uint32_t)k, t_sfa, t_sfb,
                                  (kb > 0 || k > 0) ? 1u : 0u);
                    tc_commit<2>(empty_bar + 8 * stage);   // the stage is free in both CTAs once read
                    if (++stage == kMxStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit<2>(tfull_bar);                   // accumulator complete, in both CTAs
                acc_phase ^= 1u;
            }
        }
    } else {
        // ---------------- epilogue: TMEM -> registers (all of this warp's four boxes) -> accumulator handed back ->
        // x unit -> staging -> TMA store
        const int q = warp & 3, half = (warp - 2) >> 2;
        uint8_t *buf = smem + kMxOffEpi + (warp - 2) * 4096;
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int tile = group_id; ok && tile < P.total_tiles; tile += num_groups_launched) {
            const TileInfo t = tile_info<2>(P, tile, rank);
            const int64_t m_own = t.m0 + q * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(4 * half * 32);
            uint32_t v[4][32];
            if (t.nkb > 0) {
                if (!mbar_wait_warp(tfull_bar, acc_phase, abort_flag)) { ok = false; break; }
                tc_fence_after();
                acc_phase ^= 1u;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) tc_ld32(taddr + (uint32_t)(cc * 32), v[cc]);
                tc_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(lead_tempty_bar);
            } else {
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[cc][j] = 0u;
            }
            const int32_t c_row = (int32_t)(t.m0 + q * 32), c_grp = (int32_t)(t.c_row0 / (P.M > 0 ? P.M : 1));
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const int64_t n_base = t.n0 + (4 * half + cc) * 32;
                if (n_base >= P.N || c_row >= t.row_end) continue;
                float x[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) x[j] = __uint_as_float(v[cc][j]) * X.unit;
                if (n_base + 32 > P.N && P.n_unaligned) epi_store_box_plain(P, x, t.c_row0 + m_own, n_base, m_own < t.row_end);
                else epi_store_box_tma(P, &tmC, buf, lane, x, (int32_t)n_base, c_row, c_grp);
            }
        }
        epi_store_drain(lane);
    }
    tc_teardown<2>(abort_flag, P.dev_status, tmem_base, 512, warp);
}

// ------------------------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------------------------

static size_t mx_round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static int64_t mx_pad_rows(int64_t rows) { return (rows + 255) / 256 * 256; }

size_t gemm_mx_workspace_bytes(int64_t a_rows, int64_t b_rows, int64_t K) {
    const size_t ksteps = (size_t)((K + 127) / 128);
    return mx_round_up((size_t)a_rows * K, 256) + mx_round_up((size_t)b_rows * K, 256) +
           (size_t)(mx_pad_rows(a_rows) / 128) * ksteps * kMxSfUnit + (size_t)(mx_pad_rows(b_rows) / 128) * ksteps * kMxSfUnit;
}

int gemm_mx_kernel_launches() { return 2; }

// Power-of-two scales on both operands (one per 16 or one per 32 elements); plain products and products with a grouped
// reduction (groups are multiples of 128 = whole K steps).  Row-grouped products keep the folded path.
bool gemm_mx_supported(const ufp4_qtensor *A, const ufp4_qtensor *B, int64_t M, int64_t N, int64_t K, int mode) {
    if (!is_pow2_fmt(A->scale_fmt) || !is_pow2_fmt(B->scale_fmt)) return false;
    if (mode == 1) return false;
    if (K % 16 != 0 || M < 1 || N < 1) return false;
    if (A->rows > 0x7FFFFFFF || B->rows > 0x7FFFFFFF || K > 0x7FFFFFFF) return false;
    return true;
}

static bool mx_make_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t K, int box_rows) {
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

// Scale units as a matrix of 32-bit words: one unit (512 bytes) per row, `units_per_box` consecutive units per copy.
static bool mx_make_sf_map(CUtensorMap *map, const void *ptr, int64_t units, int units_per_box) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)(kMxSfUnit / 4), (cuuint64_t)units};
    cuuint64_t strides[1] = {(cuuint64_t)kMxSfUnit};
    cuuint32_t box[2] = {(cuuint32_t)(kMxSfUnit / 4), (cuuint32_t)units_per_box};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int gemm_mx_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int mode, int64_t M,
                   int64_t N, int64_t K, const int64_t *offsets, int num_groups, int64_t group_n, void *workspace,
                   size_t workspace_bytes, int32_t *dev_status, void *stream) {
    if (!aligned_to(workspace, 256)) return UFP4_ERR_ALIGN;
    if (workspace_bytes < gemm_mx_workspace_bytes(A->rows, B->rows, K)) return UFP4_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t ksteps = (K + 127) / 128;
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    uint8_t *A8 = ws;
    uint8_t *B8 = A8 + mx_round_up((size_t)A->rows * K, 256);
    uint8_t *sfA = B8 + mx_round_up((size_t)B->rows * K, 256);
    uint8_t *sfB = sfA + (size_t)(mx_pad_rows(A->rows) / 128) * ksteps * kMxSfUnit;

    MxDecodeParams D = {};
    D.op[0] = MxOperand{static_cast<const uint8_t *>(A->codes), static_cast<const float *>(A->scales), A->ld_codes_bytes,
                        A->ld_scales, A->rows, mx_pad_rows(A->rows), codebook_of(A->grid), A8, sfA};
    D.op[1] = MxOperand{static_cast<const uint8_t *>(B->codes), static_cast<const float *>(B->scales), B->ld_codes_bytes,
                        B->ld_scales, B->rows, mx_pad_rows(B->rows), codebook_of(B->grid), B8, sfB};
    D.K = K; D.ksteps = ksteps; D.dev_status = dev_status;
    const int64_t per_row = ksteps * 4;
    D.a_ctas = (D.op[0].rows_padded * per_row + 255) / 256;
    const int64_t ctas = D.a_ctas + (D.op[1].rows_padded * per_row + 255) / 256;
    if (ctas > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    decode_mx_kernel<<<(unsigned)ctas, 256, 0, st>>>(D);
    if (cudaGetLastError() != cudaSuccess) return UFP4_ERR_CUDA;

    const int64_t a_tiles = mx_pad_rows(A->rows) / 128, b_tiles = mx_pad_rows(B->rows) / 128;
    if (ksteps * a_tiles > 0x7FFFFFFF || ksteps * b_tiles > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    CUtensorMap tmA, tmB, tmSfA, tmSfB, tmC = {};
    if (!mx_make_map(&tmA, A8, A->rows, K, kTM) || !mx_make_map(&tmB, B8, B->rows, K, kTN / 2) ||
        !mx_make_sf_map(&tmSfA, sfA, ksteps * a_tiles, 1) || !mx_make_sf_map(&tmSfB, sfB, ksteps * b_tiles, 2))
        return UFP4_ERR_CUDA;
    {
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
    P.dev_status = dev_status;
    P.mt = (int)((M + 2 * kTM - 1) / (2 * kTM));
    P.nt = (int)((N + kTN - 1) / kTN);
    const int64_t total = (int64_t)P.mt * P.nt * (mode == 2 ? num_groups : 1);
    if (total < 1 || total > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    P.total_tiles = (int)total;
    P.n_unaligned = ((N * (c_is_bf16 ? 2 : 4)) % 16) != 0;
    P.wait_limit = debug_wait_limit();
    P.skip_loads = debug_skip_loads();
    MxArgs X = {};
    X.a_tiles = a_tiles; X.b_tiles = b_tiles;
    auto unit_of = [](int grid) { return codebook_of(grid) == UFP4_GRID_INT4 ? 1.0f : (codebook_of(grid) == UFP4_GRID_E1M2 ? 0.25f : 0.5f); };
    X.unit = unit_of(A->grid) * unit_of(B->grid);

    static DeviceSetup slots[kMaxDevices];
    const DeviceSetup *dev = nullptr;
    const int rc_setup = device_setup(slots, [](int ordinal, DeviceSetup &d) -> int {
        UFP4_CUDA_OK(cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, ordinal));
        UFP4_CUDA_OK(cudaFuncSetAttribute(gemm_mx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMxSmem));
        d.max_pairs = resident_pairs(gemm_mx_kernel, kMxThreads, kMxSmem, d.num_sms);
        return UFP4_OK;
    }, &dev);
    if (rc_setup != UFP4_OK) return rc_setup;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // dependent of the decode launch above
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(2 * (unsigned)(total < dev->max_pairs ? total : dev->max_pairs));
    cfg.blockDim = dim3(kMxThreads);
    cfg.dynamicSmemBytes = kMxSmem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemm_mx_kernel, tmA, tmB, tmSfA, tmSfB, tmC, P, X) == cudaSuccess ? UFP4_OK : UFP4_ERR_CUDA;
}

}  // namespace ufp4
