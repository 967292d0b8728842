// tcgen05 / tensor-memory wrappers and the tile bookkeeping shared by the tensor-core GEMM kernels (sm_100a).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include "../../include/ufp4.h"
#include "ptx.cuh"

namespace ufp4 {

constexpr int kTM = 128, kTN = 256, kTK = 128;     // per-CTA output tile; kTK = bytes of one operand row per stage

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Completion of all MMAs issued so far by this thread -> one arrival on a barrier of this CTA (CG = 1) or on the barrier
// at the same offset in both CTAs of the pair (CG = 2: the commit is multicast to the pair; no data moves).
template <int CG>
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    if (CG == 1)
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
    else
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                     ::"r"(bar), "h"((uint16_t)3) : "memory");
}

template <int CG>
__device__ __forceinline__ void tc_mma_f8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    if (CG == 1)
        asm volatile(
            "{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p; }"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile(
            "{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p; }"
            ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

template <int CG>
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
    if (CG == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
}
template <int CG>
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    if (CG == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// Address of the same shared-memory location in another CTA of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.relaxed.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
// TMA tile load of a CTA pair: data lands in this CTA, the completion is signalled on a barrier of either CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int32_t c0, int32_t c1, uint32_t cluster_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_cta_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major, 128B-swizzled shared-memory operand: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);          // start address
    d |= (uint64_t)1u << 16;                          // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024u >> 4) << 32;                // stride byte offset between 8-row groups
    d |= (uint64_t)1u << 46;                          // descriptor version of this architecture
    d |= (uint64_t)2u << 61;                          // 128-byte swizzle
    return d;
}

// kind::f8f6f4, A = B = E5M2, D = F32, both K-major, N = 256, M = 128 (one CTA) or 256 (CTA pair).
template <int CG> struct InstrDesc {
    static constexpr uint32_t value =
        (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTN >> 3) << 17) | ((uint32_t)((kTM * CG) >> 4) << 24);
};

// ------------------------------------------------------------------------------------------------------------------
// GEMM
// ------------------------------------------------------------------------------------------------------------------

struct TcParams {
    void *C;
    int64_t ldc;
    int c_is_bf16;
    int64_t M, N, K;          // tile space M x N; K is the whole reduction length of the operands
    int mode;                 // 0 plain, 1 rows grouped, 2 reduction grouped
    const int64_t *offsets;
    int num_groups;
    int64_t group_n;
    const float *refA, *refB;
    int32_t *dev_status;
    int mt, nt, total_tiles;
    int n_unaligned;          // N * sizeof(element of C) is not a multiple of 16
    // mode 1 on CTA pairs: the 256-row tiles are laid out group by group, so that a tile never straddles two groups;
    // entry i = (first row, group) of row-tile i (a group of 128 (mod 256) rows ends with a half-filled tile)
    const int2 *mtiles;
    // quantizing epilogue (ufp4_gemm_quantized): the product, rounded to BF16, leaves as the next consumer's quantized
    // operand: blocks along N ("row" layout [M][N]) and / or blocks along M ("col" layout, stored [N][M])
    uint8_t *q_row_codes, *q_col_codes;
    float *q_row_scales, *q_col_scales;
    int64_t q_row_ldc, q_row_lds, q_col_ldc, q_col_lds;
    uint32_t q_sign_lo[8], q_sign_hi[8], q_sign[16];   // bit 31 set where eps of element 2j / 2j+1 / i of a block is -1
    int q_rht;                                          // 16-point RHT before quantizing (else none)
    // test hooks (ufp4_debug_wait_injection; both 0 in normal use): the poll limit of every bounded wait, and a mode in
    // which the TMA producer loads nothing, so that the MMA issuer's first wait runs out
    uint32_t wait_limit;
    int skip_loads;
};

// Host-side description of the quantizing epilogue's outputs (gemm_tensor_launch).
struct TcQOut {
    uint8_t *row_codes, *col_codes;
    float *row_scales, *col_scales;
    int64_t row_ldc, row_lds, col_ldc, col_lds;
    int rht, pow2;
    uint32_t sign_mask;
};

// Process-wide test hooks behind ufp4_debug_wait_injection (defined in api.cu).
uint32_t debug_wait_limit();
int debug_skip_loads();

struct TileInfo {
    int64_t m0, n0, b_row0, c_row0;
    int kb0, nkb;
    int64_t row_end;          // rows of C from here on are not this tile's to write
};

// Tile `tile` of the launch, as seen by the CTA of rank `rank` in its group of CG CTAs: the group owns a
// (CG * 128) x 256 output tile, the CTA the 128 rows [m0, m0 + 128) of it and, for CG = 2, the 128-row half
// [b_half0, b_half0 + 128) of the B tile.
template <int CG>
__device__ __forceinline__ TileInfo tile_info(const TcParams &P, int tile, int rank) {
    TileInfo t;
    const int per_group = P.mt * P.nt;
    const int g = (P.mode == 2) ? tile / per_group : 0;
    const int rem = tile - g * per_group;
    t.m0 = (int64_t)(rem / P.nt) * (kTM * CG) + (int64_t)rank * kTM;
    t.n0 = (int64_t)(rem % P.nt) * kTN;
    t.b_row0 = 0;
    t.c_row0 = 0;
    t.kb0 = 0;
    t.nkb = (int)((P.K + kTK - 1) / kTK);
    t.row_end = P.M;
    if (P.mode == 1 && CG == 2) {
        const int2 e = P.mtiles[rem / P.nt];
        t.m0 = (int64_t)e.x + (int64_t)rank * kTM;
        t.b_row0 = (int64_t)e.y * P.group_n;
        const int64_t group_end = P.offsets[e.y + 1];
        t.row_end = group_end < (int64_t)e.x + 2 * kTM ? group_end : (int64_t)e.x + 2 * kTM;
    } else if (P.mode == 1) {
        int lo = 0, hi = P.num_groups;
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (P.offsets[mid] <= t.m0) lo = mid; else hi = mid;
        }
        t.b_row0 = (int64_t)lo * P.group_n;
    } else if (P.mode == 2) {
        t.kb0 = (int)(P.offsets[g] / kTK);
        t.nkb = (int)((P.offsets[g + 1] - P.offsets[g]) / kTK);
        t.c_row0 = (int64_t)g * P.M;
    }
    return t;
}

// ------------------------------------------------------------------------------------------------------------------
// Epilogue and teardown pieces shared by the tensor-core kernels.  A warp owns a 32 x 32 box of C: lane = row of the box,
// x[j] = that row's finished value in column j.
// ------------------------------------------------------------------------------------------------------------------

// A box on the right edge whose valid part does not end on a 16-byte boundary (the TMA clips in 16-byte units): plain
// predicated stores, so that nothing right of column N is touched.  row = the lane's row of C (group offset included).
__device__ __forceinline__ void epi_store_box_plain(const TcParams &P, const float (&x)[32], int64_t row, int64_t n_base,
                                                    bool row_valid) {
    if (!row_valid) return;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (n_base + j < P.N) {
            const int64_t idx = row * P.ldc + n_base + j;
            if (P.c_is_bf16) static_cast<__nv_bfloat16 *>(P.C)[idx] = __float2bfloat16_rn(x[j]);
            else static_cast<float *>(P.C)[idx] = x[j];
        }
    }
}

// The box through the warp's staging buffer (4 KB) and one TMA store, which clips rows and columns outside C.  FP32: 128-byte
// rows in the 128B swizzle pattern (16-byte piece j of row r at piece j ^ (r & 7)); BF16: 64-byte rows in the 64B pattern
// (piece j at j ^ ((r >> 1) & 3)).  The previous box must have been read out of the buffer by its store first.
__device__ __forceinline__ void epi_store_box_tma(const TcParams &P, const CUtensorMap *tmC, uint8_t *buf, int lane,
                                                  const float (&x)[32], int32_t n_base, int32_t c_row, int32_t c_grp) {
    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
    __syncwarp();
    if (P.c_is_bf16) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t h[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                __nv_bfloat162 hh = __floats2bfloat162_rn(x[8 * j + 2 * u], x[8 * j + 2 * u + 1]);
                h[u] = *reinterpret_cast<uint32_t *>(&hh);
            }
            *reinterpret_cast<uint4 *>(buf + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
        }
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            *reinterpret_cast<float4 *>(buf + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) {
        asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                     ::"l"(tmC), "r"(n_base), "r"(c_row), "r"(c_grp), "r"(smem_u32(buf)) : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    }
}

// End of an epilogue warp's work: every box it handed to the TMA has been written.
__device__ __forceinline__ void epi_store_drain(int lane) {
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    __syncwarp();
}

// Common exit of a tensor-core kernel: all roles meet (CTA, and the pair for CG = 2, so that neither CTA leaves while the
// other may still signal its barriers); if a bounded wait gave up, copies still in flight get time to land before shared
// memory is released and UFP4_DEV_WAIT_TIMEOUT is reported; the allocating warp (warp 1) returns the tensor memory.
template <int CG>
__device__ __forceinline__ void tc_teardown(volatile uint32_t *abort_flag, int32_t *dev_status, uint32_t tmem_base,
                                            uint32_t tmem_cols, int warp) {
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();
    if (*abort_flag) {
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        if (threadIdx.x == 0 && dev_status) atomicOr(dev_status, (int)UFP4_DEV_WAIT_TIMEOUT);
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc<CG>(tmem_base, tmem_cols);
    }
}


// bf16 x bf16 -> f32 (kind::f16), one CTA, K = 16 per instruction.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

// ------------------------------------------------------------------------------------------------------------------
// Once-per-device launcher set-up (kernel attributes, SM and resident-pair counts).  Kernel attributes belong to a
// device's context, so a launcher keeps one slot per device ordinal; a slot is filled under its mutex and published
// only after every step has succeeded (a failed set-up is retried by the next call).
// ------------------------------------------------------------------------------------------------------------------
constexpr int kMaxDevices = 64;

struct DeviceSetup {
    std::mutex mu;
    std::atomic<int> ready{0};
    int num_sms = 0, max_pairs = 0;
};

// Slot of the current device, filled by init(device ordinal, slot) on first use.  Returns a ufp4_status.
template <class Init>
inline int device_setup(DeviceSetup (&slots)[kMaxDevices], Init &&init, const DeviceSetup **out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return UFP4_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return UFP4_ERR_UNSUPPORTED;
    DeviceSetup &d = slots[dev];
    if (!d.ready.load(std::memory_order_acquire)) {
        std::lock_guard<std::mutex> lock(d.mu);
        if (!d.ready.load(std::memory_order_relaxed)) {
            const int rc = init(dev, d);
            if (rc != UFP4_OK) return rc;
            d.ready.store(1, std::memory_order_release);
        }
    }
    *out = &d;
    return UFP4_OK;
}

// How many CTA pairs (clusters of 2) of `kernel` can be resident at once; an SM whose neighbour is unavailable cannot
// host half a pair.
template <class Kernel>
inline int resident_pairs(Kernel kernel, int threads, int smem_bytes, int num_sms) {
    cudaLaunchConfig_t probe = {};
    cudaLaunchAttribute pattr[1];
    pattr[0].id = cudaLaunchAttributeClusterDimension;
    pattr[0].val.clusterDim.x = 2; pattr[0].val.clusterDim.y = 1; pattr[0].val.clusterDim.z = 1;
    probe.gridDim = dim3(2 * (num_sms / 2)); probe.blockDim = dim3(threads); probe.dynamicSmemBytes = smem_bytes;
    probe.attrs = pattr; probe.numAttrs = 1;
    int pairs = 0;
    if (cudaOccupancyMaxActiveClusters(&pairs, kernel, &probe) != cudaSuccess || pairs < 1) pairs = num_sms / 2;
    return pairs;
}

}  // namespace ufp4
