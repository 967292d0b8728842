// Native-FP4 tensor-core path for operands with E4M3 block scales x a per-tensor FP32 scale (the two-level hierarchy
// Sec. 2.1's footnote attributes to NVFP4; Sec. 2.2: Y^ = Q_G(XH') Q_G(WH')^T): tcgen05.mma kind::mxf4nvf4 with one
// UE4M3 scale per 16 elements of K and operand row, applied by the tensor core.
//
// The FP4 tensor path knows the E2M1 levels only (the paper's premise, Sec. 1).  An E2M1-grid tensor is its operand as it
// stands: its packed codes are read by TMA directly.  A uniform code q in [-8, 7] is the sum of two E2M1 values in half
// units, q / 2 = hi + lo with hi in {0, .5, 1, 1.5, 2, 3, 4} and lo in {0, .5} (|q| = 5 -> 2 + .5, |q| = 7 -> 3 + .5),
// both with q's sign, so A B^T = (Ah + Al)(Bh + Bl)^T is four MMAs per K step on two planes per operand (two when one
// operand is an E2M1 tensor, one when both are).  FP4 MMAs run at twice the 8-bit rate, so the uniform x uniform product
// has the ceiling of one FP16 MMA per K step; it moves half the operand bytes.  The two tensor scales and the grids' code
// units multiply the result once in the epilogue (they enter the definition as RN(ts x E4M3 value): a relative 2^-24
// per operand).  Two kernels:
//   1. decode_nvf4_kernel: uniform nibbles -> hi and lo planes [rows][K / 2]; E4M3 scale bytes -> the 512-byte units the
//      tensor core's scale copy takes (unit = 128 rows x the 4 blocks of a 64-element MMA step, byte of row r, block j at
//      (r % 32) * 16 + (r / 32) * 4 + j), stored [K stage of 256][row tile][step].
//   2. gemm_nvf4_kernel<PA, PB>: persistent, warp-specialised, one CTA pair per 256 x 256 tile, K stage = 256 elements
//      (128 bytes per row and plane).  Each CTA's producer brings its rows of every plane and the scale units by TMA; the
//      leader's MMA thread copies a stage's scales to tensor memory (tcgen05.cp.cta_group::2: 16 columns for A, 32 for
//      B) and issues PA x PB block-scaled MMAs (M256 x N256 x K64) per 64-element step.  One 256-column accumulator
//      (the scale columns leave no room for a second): the epilogue warps drain it into registers, hand it back and
//      then store C through their staging buffers and TMA stores (a whole 32 x 32 box at a time, or half a box where two
//      planes per operand leave the ring only 2 KB per warp).
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdlib.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tc.cuh"

namespace ufp4 {

constexpr int kNvKStage = 256;                        // elements of K per stage
constexpr int kNvPlane = kTM * kTK;                   // 16 KB: 128 rows x 128 bytes of packed nibbles
constexpr int kNvSfUnit = 512;
constexpr int kNvSfA = 4 * kNvSfUnit, kNvSfB = 8 * kNvSfUnit;     // own rows of A; all 256 rows of the B tile
constexpr int kNvEpiWarps = 8;
constexpr int kNvThreads = 64 + 32 * kNvEpiWarps;
constexpr int kNvBarBytes = 256;
constexpr int kNvMaxSmem = 227 * 1024;

template <int PA, int PB> struct NvCfg {
    static constexpr int kStageBytes = (PA + PB) * kNvPlane + kNvSfA + kNvSfB;      // a multiple of 1024
    // C leaves through one staging buffer per epilogue warp and TMA stores: a whole 32 x 32 box (4 KB for FP32) where the
    // ring leaves room, half a box at a time (2 KB) with two planes per operand
    static constexpr int kEpiPerWarp = PA + PB <= 3 ? 4096 : 2048;
    static constexpr int kEpiBytes = kNvEpiWarps * kEpiPerWarp;
    static constexpr int kFit = (kNvMaxSmem - kNvBarBytes - kEpiBytes) / kStageBytes;
    static constexpr int kStages = kFit > 6 ? 6 : kFit;
    static constexpr int kOffEpi = kStages * kStageBytes;
    static constexpr int kOffBars = kOffEpi + kEpiBytes;
    static constexpr int kSmem = kOffBars + kNvBarBytes;
    static_assert(kStageBytes % 1024 == 0 && kStages >= 3 && kSmem <= kNvMaxSmem, "operand ring");
    static_assert(16 * kStages + 24 <= 160, "barriers, the tensor-memory slot and the abort flag share 256 bytes");
};

// ------------------------------------------------------------------------------------------------------------------
// decode
// ------------------------------------------------------------------------------------------------------------------

struct NvOperand {
    const uint8_t *codes;
    const uint8_t *scales;                 // E4M3 bytes [rows][lds]
    int64_t ldc, lds, rows, rows_padded;   // rows_padded: multiple of 256 (whole scale units for every tile)
    int grid;                              // codebook
    uint8_t *hi, *lo;                      // planes [rows][pitch] (uniform grids only)
    uint8_t *sf;                           // [kstages][rows_padded / 128][4][512]
};

struct NvDecodeParams {
    NvOperand op[2];
    int64_t K, kstages, pitch;             // kstages = ceil(K / 256); pitch = K / 2 rounded up to 16 bytes
    int64_t a_threads;
};

// Eight nibbles of uniform codes -> the E2M1 nibbles of hi and lo.
__device__ __forceinline__ void split_uniform8(uint32_t w, bool int4, uint32_t *hi, uint32_t *lo) {
    uint32_t is8 = 0u;
    if (int4) {
        // two's complement -> sign | magnitude; -8 (never written by the quantizer) is taken out first: it becomes hi = -4
        const uint32_t t = w ^ 0x88888888u;
        const uint32_t nz = (((t & 0x77777777u) + 0x77777777u) | t) & 0x88888888u;       // bit 3 set where nibble != 8
        is8 = ~nz & 0x88888888u;
        w &= ~((is8 >> 3) * 0xFu);
        const uint32_t m = (w & 0x88888888u) >> 3;
        w = (w ^ (m * 7u)) + m;
    }
    const uint32_t S = w & 0x88888888u;
    const uint32_t B2 = (w >> 2) & 0x11111111u, B1 = (w >> 1) & 0x11111111u, B0 = w & 0x11111111u;
    const uint32_t lo1 = B2 & B0;                                                         // magnitudes 5 and 7 carry a half
    *lo = lo1 | ((lo1 << 3) & S);
    // magnitude m < 4: the E2M1 code of m / 2 is m itself; 4, 5 -> code 4 (2.0); 6, 7 -> code 5 (3.0)
    *hi = (w & 0x44444444u) | (B2 & B1) | (~(B2 * 3u) & w & 0x33333333u) | S | ((is8 >> 3) * 0xEu);
}

// One thread per (row, 64-element MMA step): 32 bytes of codes -> 32 + 32 bytes of planes, 4 scale bytes -> one word of a unit.
__global__ void __launch_bounds__(256) decode_nvf4_kernel(const NvDecodeParams P) {
    // the product kernel of the same call is a programmatic dependent launch: see its griddepcontrol.wait
    asm volatile("griddepcontrol.launch_dependents;");
    const int64_t gid0 = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const bool is_b = gid0 >= P.a_threads;
    const NvOperand &O = P.op[is_b ? 1 : 0];
    const int64_t gid = gid0 - (is_b ? P.a_threads : 0);
    const int64_t nsteps = P.kstages * 4;
    const int64_t row = gid / nsteps, c = gid - row * nsteps;
    if (row >= O.rows_padded) return;
    uint32_t *sf = reinterpret_cast<uint32_t *>(O.sf + ((((c >> 2) * (O.rows_padded >> 7) + (row >> 7)) << 2) + (c & 3)) * kNvSfUnit +
                                                ((row & 31) << 4) + (((row >> 5) & 3) << 2));
    const int64_t nkb = P.K >> 4;
    if (row >= O.rows || 4 * c >= nkb) {
        *sf = 0u;                            // padding: scale 0 on all-zero elements (the TMA fills those with zeros)
        return;
    }
    uint32_t sw = 0u;
    const uint8_t *sp = O.scales + row * O.lds + 4 * c;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (4 * c + j < nkb) sw |= (uint32_t)__ldg(sp + j) << (8 * j);
    *sf = sw;
    if (O.hi == nullptr) return;             // E2M1 tensors: the product kernel reads their codes in place
    const bool int4 = O.grid == UFP4_GRID_INT4;
    const uint8_t *cp = O.codes + row * O.ldc + 32 * c;
    uint8_t *hp = O.hi + row * P.pitch + 32 * c, *lp = O.lo + row * P.pitch + 32 * c;
    if (4 * c + 4 <= nkb) {
        // a whole step: two 16-byte loads, two 16-byte stores per plane (rows and steps are 16-byte aligned)
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const uint4 w = __ldg(reinterpret_cast<const uint4 *>(cp) + j);
            uint4 h, l;
            split_uniform8(w.x, int4, &h.x, &l.x);
            split_uniform8(w.y, int4, &h.y, &l.y);
            split_uniform8(w.z, int4, &h.z, &l.z);
            split_uniform8(w.w, int4, &h.w, &l.w);
            reinterpret_cast<uint4 *>(hp)[j] = h;
            reinterpret_cast<uint4 *>(lp)[j] = l;
        }
        return;
    }
    for (int j = 0; 4 * c + j < nkb; ++j) {          // the last step of a row whose K is not a multiple of 64
        const uint2 w = __ldg(reinterpret_cast<const uint2 *>(cp) + j);
        uint2 h, l;
        split_uniform8(w.x, int4, &h.x, &l.x);
        split_uniform8(w.y, int4, &h.y, &l.y);
        reinterpret_cast<uint2 *>(hp)[j] = h;
        reinterpret_cast<uint2 *>(lp)[j] = l;
    }
}

// ------------------------------------------------------------------------------------------------------------------
// product
// ------------------------------------------------------------------------------------------------------------------

__device__ __forceinline__ uint64_t nv_sf_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)1u << 16;
    d |= (uint64_t)(128u >> 4) << 32;
    d |= (uint64_t)1u << 46;
    return d;
}
// One scale unit from shared to tensor memory in both CTAs of the pair (each from its own shared memory into its own
// tensor memory): 4 columns.
__device__ __forceinline__ void nv_cp_sf(uint32_t taddr, uint64_t desc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(desc) : "memory");
}
// kind::mxf4nvf4, block-scaled, on a CTA pair: A = B = E2M1 (format 1), UE4M3 scales (format bit clear), both K-major,
// M = 256, N = 256, K = 64; the four bytes of a scale column entry are the four 16-element blocks of the step.
__device__ __forceinline__ void nv_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t t_sfa, uint32_t t_sfb,
                                       uint32_t accumulate) {
    constexpr uint32_t idesc = (1u << 7) | (1u << 10) | ((uint32_t)(kTN >> 3) << 17) | ((uint32_t)((2 * kTM) >> 4) << 24);
    asm volatile(
        "{ .reg .pred p; setp.ne.b32 p, %6, 0; "
        "tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.scale_vec::4X [%0], %1, %2, %3, [%4], [%5], p; }"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(t_sfa), "r"(t_sfb), "r"(accumulate) : "memory");
}

struct NvMaps {
    CUtensorMap a[2], b[2], sfa, sfb, c;     // c: boxes of 32 columns x 32 rows, or x 16 rows for FP32 with 2 KB staging buffers
};

struct NvArgs {
    int64_t a_tiles, b_tiles;    // 128-row tiles of the (padded) scale arrays
    const float *tsA, *tsB;      // the two tensor scales (device)
    float unit;                  // product of the grids' code units in the planes' half units
};

// A warp's 32 x 32 FP32 box through a 2 KB staging buffer: rows 0..15, then rows 16..31, each as a 16 x 32 box in the
// 128B swizzle pattern (16-byte piece j of row r at piece j ^ (r & 7)) handed to one TMA store, which clips at M and N.
__device__ __forceinline__ void nv_store_box_halves(const CUtensorMap *tmC, uint8_t *buf, int lane, const float (&x)[32],
                                                    int32_t n_base, int32_t c_row) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
        if ((lane >> 4) == h) {
            const int r = lane & 15;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                *reinterpret_cast<float4 *>(buf + r * 128 + ((j ^ (r & 7)) << 4)) = make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
            asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                         ::"l"(tmC), "r"(n_base), "r"(c_row + 16 * h), "r"(0), "r"(smem_u32(buf)) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
    }
}

template <int PA, int PB>
__global__ void __launch_bounds__(kNvThreads, 1)
gemm_nvf4_kernel(const __grid_constant__ NvMaps M, const TcParams P, const NvArgs X) {
    using Cfg = NvCfg<PA, PB>;
    constexpr int kStages = Cfg::kStages, kStageBytes = Cfg::kStageBytes;
    constexpr int kOffB = PA * kNvPlane, kOffSfA = (PA + PB) * kNvPlane, kOffSfB = kOffSfA + kNvSfA;
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = smem_u32(smem);
    const uint32_t bars = base + Cfg::kOffBars;
    const uint32_t full_bar = bars, empty_bar = bars + 8 * kStages, tfull_bar = bars + 16 * kStages, tempty_bar = tfull_bar + 8;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + Cfg::kOffBars + 16 * kStages + 16);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(smem + Cfg::kOffBars + 160);   // flag, poll limit
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // rank 0 of the pair issues the MMAs and owns the barriers the pair synchronises on
    const int rank = (int)cluster_cta_rank();
    const int group_id = blockIdx.x / 2, num_groups_launched = gridDim.x / 2;
    const uint32_t lead_full_bar = map_to_cta(full_bar, 0), lead_tempty_bar = map_to_cta(tempty_bar, 0);
    const int nks = (int)((P.K + kNvKStage - 1) / kNvKStage);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar + 8 * s, 2);              // one arrive.expect_tx per CTA of the pair
            mbar_init(empty_bar + 8 * s, 1);
        }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, 2 * kNvEpiWarps);
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
    const uint32_t t_sfa = tmem_base + kTN, t_sfb = tmem_base + kTN + 16;    // accumulator: columns 0..255, then the scales

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer: this CTA's rows of every plane, the scales of its A rows and of the whole B tile
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = group_id; ok && !P.skip_loads && tile < P.total_tiles; tile += num_groups_launched) {
                const TileInfo t = tile_info<2>(P, tile, rank);
                const int32_t ta = (int32_t)(t.m0 >> 7), tb = (int32_t)(t.n0 >> 7);
                for (int ks = 0; ks < nks; ++ks) {
                    if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t fb = lead_full_bar + 8 * stage, st = base + stage * kStageBytes;
                    if (rank == 0) mbar_expect_tx(full_bar + 8 * stage, kStageBytes);
                    else mbar_expect_tx_cluster(fb, kStageBytes);
#pragma unroll
                    for (int p = 0; p < PA; ++p) tma_load_2d_pair(st + p * kNvPlane, &M.a[p], ks * kTK, (int32_t)t.m0, fb);
#pragma unroll
                    for (int p = 0; p < PB; ++p)
                        tma_load_2d_pair(st + kOffB + p * kNvPlane, &M.b[p], ks * kTK, (int32_t)(t.n0 + rank * (kTN / 2)), fb);
                    tma_load_2d_pair(st + kOffSfA, &M.sfa, 0, (int32_t)(((int64_t)ks * X.a_tiles + ta) * 4), fb);
                    tma_load_2d_pair(st + kOffSfB, &M.sfb, 0, (int32_t)(((int64_t)ks * X.b_tiles + tb) * 4), fb);
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
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
                if (!mbar_wait(tempty_bar, acc_phase ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                for (int ks = 0; ks < nks; ++ks) {
                    if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t st = base + stage * kStageBytes;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        nv_cp_sf(t_sfa + 4 * c, nv_sf_desc(st + kOffSfA + c * kNvSfUnit));
                        nv_cp_sf(t_sfb + 8 * c, nv_sf_desc(st + kOffSfB + c * kNvSfUnit));
                        nv_cp_sf(t_sfb + 8 * c + 4, nv_sf_desc(st + kOffSfB + (4 + c) * kNvSfUnit));
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
#pragma unroll
                        for (int pa = 0; pa < PA; ++pa) {
#pragma unroll
                            for (int pb = 0; pb < PB; ++pb) {
                                // advancing K inside the 128-byte swizzle span: 64 elements = 32 bytes = +2 in the (address >> 4) field
                                nv_mma(tmem_base, umma_desc_sw128(st + pa * kNvPlane) + (uint64_t)(2 * c),
                                       umma_desc_sw128(st + kOffB + pb * kNvPlane) + (uint64_t)(2 * c), t_sfa + 4 * c, t_sfb + 8 * c,
                                       (ks > 0 || c > 0 || pa > 0 || pb > 0) ? 1u : 0u);
                            }
                        }
                    }
                    tc_commit<2>(empty_bar + 8 * stage);   // the stage is free in both CTAs once read
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                tc_commit<2>(tfull_bar);                   // accumulator complete, in both CTAs
                acc_phase ^= 1u;
            }
        }
    } else {
        // ---------------- epilogue: TMEM -> registers (all of this warp's four boxes) -> accumulator handed back ->
        // x tensor scales and code units -> global memory
        const int q = warp & 3, half = (warp - 2) >> 2;
        uint8_t *buf = smem + Cfg::kOffEpi + (warp - 2) * Cfg::kEpiPerWarp;
        const float scale = __fmul_rn(__fmul_rn(__ldg(X.tsA), __ldg(X.tsB)), X.unit);
        uint32_t acc_phase = 0;
        bool ok = true;
        for (int tile = group_id; ok && tile < P.total_tiles; tile += num_groups_launched) {
            const TileInfo t = tile_info<2>(P, tile, rank);
            const int64_t m_own = t.m0 + q * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(4 * half * 32);
            uint32_t v[4][32];
            if (!mbar_wait_warp(tfull_bar, acc_phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            acc_phase ^= 1u;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) tc_ld32(taddr + (uint32_t)(cc * 32), v[cc]);
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(lead_tempty_bar);
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const int64_t n_base = t.n0 + (4 * half + cc) * 32;
                if (n_base >= P.N) continue;
                float x[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) x[j] = __uint_as_float(v[cc][j]) * scale;
                const int32_t c_row = (int32_t)(t.m0 + q * 32);
                if (c_row >= t.row_end) continue;
                if (n_base + 32 > P.N && P.n_unaligned) epi_store_box_plain(P, x, m_own, n_base, m_own < t.row_end);
                else if (Cfg::kEpiPerWarp == 4096 || P.c_is_bf16) epi_store_box_tma(P, &M.c, buf, lane, x, (int32_t)n_base, c_row, 0);
                else nv_store_box_halves(&M.c, buf, lane, x, (int32_t)n_base, c_row);
            }
        }
        epi_store_drain(lane);
    }
    tc_teardown<2>(abort_flag, P.dev_status, tmem_base, 512, warp);
}

// ------------------------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------------------------

static size_t nv_round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static int64_t nv_pad_rows(int64_t rows) { return (rows + 255) / 256 * 256; }
static bool nv_uniform(const ufp4_qtensor *T) { return codebook_of(T->grid) != UFP4_GRID_E2M1; }
static size_t nv_plane_bytes(const ufp4_qtensor *T) {
    return nv_uniform(T) ? nv_round_up((size_t)T->rows * nv_round_up((size_t)T->k / 2, 16), 256) : 0;
}
static size_t nv_sf_bytes(const ufp4_qtensor *T) {
    return (size_t)((T->k + kNvKStage - 1) / kNvKStage) * (size_t)(nv_pad_rows(T->rows) / 128) * 4 * kNvSfUnit;
}

size_t gemm_nvf4_workspace_bytes(const ufp4_qtensor *A, const ufp4_qtensor *B) {
    return 2 * nv_plane_bytes(A) + 2 * nv_plane_bytes(B) + nv_sf_bytes(A) + nv_sf_bytes(B);
}

int gemm_nvf4_kernel_launches() { return 2; }

// Both operands with E4M3 block scales x a tensor scale; plain products.
bool gemm_nvf4_supported(const ufp4_qtensor *A, const ufp4_qtensor *B, int64_t M, int64_t N, int64_t K, int mode) {
    if (A->scale_fmt != UFP4_SCALE_E4M3_TENSOR || B->scale_fmt != UFP4_SCALE_E4M3_TENSOR) return false;
    if (mode != 0) return false;
    if (K % 16 != 0 || M < 1 || N < 1) return false;
    if (A->rows > 0x7FFFFFFF || B->rows > 0x7FFFFFFF || K > 0x7FFFFFFF) return false;
    return true;
}

static bool nv_make_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t k_bytes, int64_t pitch) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)k_bytes, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)pitch};
    cuuint32_t box[2] = {(cuuint32_t)kTK, (cuuint32_t)kTM};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Scale units as a matrix of 32-bit words: one unit (512 bytes) per row, `units_per_box` consecutive units per copy.
static bool nv_make_sf_map(CUtensorMap *map, const void *ptr, int64_t units, int units_per_box) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)(kNvSfUnit / 4), (cuuint64_t)units};
    cuuint64_t strides[1] = {(cuuint64_t)kNvSfUnit};
    cuuint32_t box[2] = {(cuuint32_t)(kNvSfUnit / 4), (cuuint32_t)units_per_box};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int PA, int PB>
static int nv_launch(const NvMaps &maps, const TcParams &P, const NvArgs &X, int64_t total, cudaStream_t st) {
    using Cfg = NvCfg<PA, PB>;
    static DeviceSetup slots[kMaxDevices];
    const DeviceSetup *dev = nullptr;
    const int rc_setup = device_setup(slots, [](int ordinal, DeviceSetup &d) -> int {
        UFP4_CUDA_OK(cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, ordinal));
        UFP4_CUDA_OK(cudaFuncSetAttribute(gemm_nvf4_kernel<PA, PB>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmem));
        d.max_pairs = resident_pairs(gemm_nvf4_kernel<PA, PB>, kNvThreads, Cfg::kSmem, d.num_sms);
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
    cfg.blockDim = dim3(kNvThreads);
    cfg.dynamicSmemBytes = Cfg::kSmem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemm_nvf4_kernel<PA, PB>, maps, P, X) == cudaSuccess ? UFP4_OK : UFP4_ERR_CUDA;
}

int gemm_nvf4_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int64_t M, int64_t N,
                     int64_t K, void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream) {
    if (!aligned_to(workspace, 256)) return UFP4_ERR_ALIGN;
    if (workspace_bytes < gemm_nvf4_workspace_bytes(A, B)) return UFP4_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t kstages = (K + kNvKStage - 1) / kNvKStage;
    const int64_t pitch = (int64_t)nv_round_up((size_t)K / 2, 16);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    uint8_t *planes[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};
    const ufp4_qtensor *T[2] = {A, B};
    for (int o = 0; o < 2; ++o) {
        const size_t pb = nv_plane_bytes(T[o]);
        if (pb) {
            planes[o][0] = ws; ws += pb;
            planes[o][1] = ws; ws += pb;
        }
    }
    uint8_t *sf[2];
    sf[0] = ws; ws += nv_sf_bytes(A);
    sf[1] = ws;

    NvDecodeParams D = {};
    for (int o = 0; o < 2; ++o)
        D.op[o] = NvOperand{static_cast<const uint8_t *>(T[o]->codes), static_cast<const uint8_t *>(T[o]->scales),
                            T[o]->ld_codes_bytes, T[o]->ld_scales, T[o]->rows, nv_pad_rows(T[o]->rows), codebook_of(T[o]->grid),
                            planes[o][0], planes[o][1], sf[o]};
    D.K = K; D.kstages = kstages; D.pitch = pitch;
    D.a_threads = (D.op[0].rows_padded * kstages * 4 + 255) / 256 * 256;
    const int64_t ctas = (D.a_threads + D.op[1].rows_padded * kstages * 4 + 255) / 256;
    if (ctas > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    decode_nvf4_kernel<<<(unsigned)ctas, 256, 0, st>>>(D);
    if (cudaGetLastError() != cudaSuccess) return UFP4_ERR_CUDA;

    const int64_t a_tiles = nv_pad_rows(A->rows) / 128, b_tiles = nv_pad_rows(B->rows) / 128;
    if (kstages * a_tiles * 4 > 0x7FFFFFFF || kstages * b_tiles * 4 > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    NvMaps maps = {};
    const int pa = nv_uniform(A) ? 2 : 1, pb = nv_uniform(B) ? 2 : 1;
    for (int o = 0; o < 2; ++o) {
        CUtensorMap *m = o == 0 ? maps.a : maps.b;
        if (nv_uniform(T[o])) {
            if (!nv_make_map(&m[0], planes[o][0], T[o]->rows, K / 2, pitch) || !nv_make_map(&m[1], planes[o][1], T[o]->rows, K / 2, pitch))
                return UFP4_ERR_CUDA;
        } else {
            if (!nv_make_map(&m[0], T[o]->codes, T[o]->rows, K / 2, T[o]->ld_codes_bytes)) return UFP4_ERR_CUDA;
            m[1] = m[0];
        }
    }
    if (!nv_make_sf_map(&maps.sfa, sf[0], kstages * a_tiles * 4, 4) || !nv_make_sf_map(&maps.sfb, sf[1], kstages * b_tiles * 4, 8))
        return UFP4_ERR_CUDA;
    {
        // C as [1][rows][cols] for the staged epilogue's TMA stores, which clip at M and N
        EncodeTiledFn fn = encode_tiled_fn();
        if (!fn) return UFP4_ERR_CUDA;
        const cuuint64_t es = c_is_bf16 ? 2 : 4;
        cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)M, 1};
        cuuint64_t strides[2] = {(cuuint64_t)ldc * es, (cuuint64_t)M * (cuuint64_t)ldc * es};
        cuuint32_t box[3] = {32, (cuuint32_t)((pa + pb <= 3 || c_is_bf16) ? 32 : 16), 1};
        cuuint32_t estr[3] = {1, 1, 1};
        if (fn(&maps.c, c_is_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, C, dims, strides, box,
               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, c_is_bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return UFP4_ERR_CUDA;
    }

    TcParams P = {};
    P.C = C; P.ldc = ldc; P.c_is_bf16 = c_is_bf16;
    P.M = M; P.N = N; P.K = K; P.mode = 0;
    P.dev_status = dev_status;
    P.mt = (int)((M + 2 * kTM - 1) / (2 * kTM));
    P.nt = (int)((N + kTN - 1) / kTN);
    const int64_t total = (int64_t)P.mt * P.nt;
    if (total < 1 || total > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    P.total_tiles = (int)total;
    P.n_unaligned = ((N * (c_is_bf16 ? 2 : 4)) % 16) != 0;
    P.wait_limit = debug_wait_limit();
    P.skip_loads = debug_skip_loads();
    NvArgs X = {};
    X.a_tiles = a_tiles; X.b_tiles = b_tiles;
    X.tsA = A->tensor_scale; X.tsB = B->tensor_scale;
    // planes hold q / 2 for the uniform grids (INT4: value q, E1M2: value q / 4) and the level itself for E2M1
    auto unit_of = [](int grid) { return codebook_of(grid) == UFP4_GRID_INT4 ? 2.0f : (codebook_of(grid) == UFP4_GRID_E1M2 ? 0.5f : 1.0f); };
    X.unit = unit_of(A->grid) * unit_of(B->grid);
    if (pa == 2 && pb == 2) return nv_launch<2, 2>(maps, P, X, total, st);
    if (pa == 2) return nv_launch<2, 1>(maps, P, X, total, st);
    if (pb == 2) return nv_launch<1, 2>(maps, P, X, total, st);
    return nv_launch<1, 1>(maps, P, X, total, st);
}

}  // namespace ufp4
