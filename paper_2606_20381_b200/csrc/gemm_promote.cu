// Tensor-core path of the block-scaled 4-bit GEMM (Sec. 2.2: Y^ = Q_G(XH') Q_G(WH')^T) for arbitrary FP32 block scales
// (Table 1's "FP32 single-level" scale, and the E4M3 x tensor two-level format).
//
// code x FP32 scale needs up to 27 significant bits, so it cannot be folded into any single tensor-core operand (the
// split path carries it as two FP16 pieces and is the faster of the two; this path is taken on request).  Here the
// integer codes go to the tensor cores and the scales to the CUDA cores: per 16-element quant block one
// tcgen05.mma kind::f16 (K = 16, BF16 operands holding the exact integers q, FP32 accumulation, no carry-in) writes the
// exact integer partial P_kb[m][n] of a 128 x 128 tile into tensor memory, and eight "promotion" warps read it back
// (tcgen05.ld) and accumulate acc[m][n] += P_kb[m][n] * (sA[m][kb] * sB[n][kb]) in registers with packed FP32 FMAs.
// The promotion is M*N*K/16 multiply-adds on the CUDA cores and bounds this path at a fraction of the tensor peak; the
// tensor cores replace the integer dot products of the plain exact kernel, which is what made that kernel slow.
//   1. decode_promote_kernel: packed nibbles -> BF16 integers [rows][K]; scales -> FP32, transposed to [K/16][rows] so that
//      a stage's scales land in shared memory as contiguous per-block rows (caller's workspace).
//   2. gemm_promote_kernel: persistent; warp 0 TMA producer (4-stage ring: A, B, sA, sB), warp 1 MMA issuer (one MMA per
//      quant block into four alternating 128-column tensor-memory buffers), warps 2-9 promotion + epilogue (TMA stores).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp8.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tc.cuh"

namespace ufp4 {

constexpr int kPN = 128;                            // tile is 128 x 128
constexpr int kPKElems = 64;                        // K elements per stage (128 bytes of BF16): 4 quant blocks
constexpr int kPStages = 4;
constexpr int kPBufs = 4;                           // partial-product buffers in tensor memory (128 columns each)
constexpr int kPOperandStage = kTM * 128;           // 16 KB per operand per stage
constexpr int kPScaleStage = 4 * kTM * 4;           // 4 blocks x 128 rows x FP32 = 2 KB per operand per stage
constexpr int kPThreads = 64 + 32 * 8;
constexpr int kPOffB = kPStages * kPOperandStage;
constexpr int kPOffSA = 2 * kPStages * kPOperandStage;
constexpr int kPOffSB = kPOffSA + kPStages * kPScaleStage;
constexpr int kPOffEpi = kPOffSB + kPStages * kPScaleStage;      // 8 warps x 4 KB staging (1024-aligned)
constexpr int kPOffBars = kPOffEpi + 8 * 4096;
constexpr int kPSmem = kPOffBars + 256;
constexpr uint32_t kPStageTx = 2 * kPOperandStage + 2 * kPScaleStage;
static_assert(kPOffEpi % 1024 == 0, "staging buffers must keep the swizzle alignment");

// ------------------------------------------------------------------------------------------------------------------
// decode: nibbles -> BF16 integers, scales -> transposed FP32
// ------------------------------------------------------------------------------------------------------------------

struct PDecodeOperand {
    const uint8_t *codes;
    const void *scales;
    const float *tensor_scale;
    int64_t ldc, lds, rows, ldt;   // ldt: row pitch (in floats) of the transposed scale array
    int grid, sfmt;
    __nv_bfloat16 *out16;          // [rows][K]
    float *scales_t;               // [K/16][ldt]
};

struct PDecodeParams {
    PDecodeOperand op[2];
    int64_t K, a_ctas;
};

__global__ void __launch_bounds__(256) decode_promote_kernel(const PDecodeParams P) {
    const bool is_b = (int64_t)blockIdx.x >= P.a_ctas;
    const PDecodeOperand &O = P.op[is_b ? 1 : 0];
    const int lane = threadIdx.x & 31;
    const int64_t row = ((int64_t)blockIdx.x - (is_b ? P.a_ctas : 0)) * 8 + (threadIdx.x >> 5);
    if (row >= O.rows) return;
    const int nkb = (int)(P.K >> 4);
    // value of a code = integer stored here x unit: INT4 q, E1M2 q/4, E2M1 (2 value)/2
    const float unit = O.grid == UFP4_GRID_INT4 ? 1.0f : (O.grid == UFP4_GRID_E1M2 ? 0.25f : 0.5f);
    const float ts = O.sfmt == UFP4_SCALE_E4M3_TENSOR ? *O.tensor_scale : 1.0f;
    const uint2 *cptr = reinterpret_cast<const uint2 *>(O.codes + row * O.ldc);
    uint4 *optr = reinterpret_cast<uint4 *>(O.out16 + row * P.K);
    for (int kb = lane; kb < nkb; kb += 32) {
        float s;
        if (O.sfmt == UFP4_SCALE_E4M3_TENSOR) {
            const uint8_t byte = static_cast<const uint8_t *>(O.scales)[row * O.lds + kb];
            __half_raw hr = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)byte, __NV_E4M3);
            s = __fmul_rn(ts, __half2float(*reinterpret_cast<__half *>(&hr)));
        } else {
            s = static_cast<const float *>(O.scales)[row * O.lds + kb];
        }
        O.scales_t[(int64_t)kb * O.ldt + row] = s * unit;
        const uint2 cw = __ldg(cptr + kb);
        uint32_t out[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t pair = 0;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int e = 2 * j + h;
                const uint32_t nib = ((e < 8 ? cw.x : cw.y) >> (4 * (e & 7))) & 0xFu;
                int q;
                if (O.grid == UFP4_GRID_INT4) q = (int)(nib ^ 8u) - 8;
                else {
                    int mag = nib & 7;
                    if (O.grid == UFP4_GRID_E2M1) mag = mag < 2 ? mag : (2 + (mag & 1)) << ((mag >> 1) - 1);
                    q = (nib & 8u) ? -mag : mag;
                }
                __nv_bfloat16 b = __float2bfloat16_rn((float)q);       // |q| <= 12: exact
                pair |= (uint32_t)(*reinterpret_cast<unsigned short *>(&b)) << (16 * h);
            }
            out[j] = pair;
        }
        // one 32-byte store per block (rows are 32-byte aligned: K is a multiple of 16)
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     :: "l"(optr + 2 * kb), "r"(out[0]), "r"(out[1]), "r"(out[2]), "r"(out[3]), "r"(out[4]), "r"(out[5]), "r"(out[6]), "r"(out[7])
                     : "memory");
    }
}

// Packed FP32 pairs (explicitly rounded; used for the promotion).
__device__ __forceinline__ float2 pmul2(float2 a, float2 b) {
    float2 d;
    asm("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mul.rn.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float2 pfma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{ .reg .b64 ra, rb, rc, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mov.b64 rc, {%6, %7}; "
        "fma.rn.f32x2 rd, ra, rb, rc; mov.b64 {%0, %1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}

struct PTile {
    int64_t m0, n0, b_row0, c_row0;
    int ks0, nks;     // first stage index along K (in units of 64 elements) and number of stages
};

__device__ __forceinline__ PTile ptile_info(const TcParams &P, int tile) {
    PTile t;
    const int per_group = P.mt * P.nt;
    const int g = (P.mode == 2) ? tile / per_group : 0;
    const int rem = tile - g * per_group;
    t.m0 = (int64_t)(rem / P.nt) * kTM;
    t.n0 = (int64_t)(rem % P.nt) * kPN;
    t.b_row0 = 0;
    t.c_row0 = 0;
    t.ks0 = 0;
    t.nks = (int)((P.K + kPKElems - 1) / kPKElems);
    if (P.mode == 1) {
        int lo = 0, hi = P.num_groups;
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (P.offsets[mid] <= t.m0) lo = mid; else hi = mid;
        }
        t.b_row0 = (int64_t)lo * P.group_n;
    } else if (P.mode == 2) {
        t.ks0 = (int)(P.offsets[g] / kPKElems);
        t.nks = (int)((P.offsets[g + 1] - P.offsets[g]) / kPKElems);
        t.c_row0 = (int64_t)g * P.M;
    }
    return t;
}

// kind::f16, A = B = BF16, D = F32, both K-major, M = 128, N = 128.
constexpr uint32_t kPInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kPN >> 3) << 17) | ((uint32_t)(kTM >> 4) << 24);

__global__ void __launch_bounds__(kPThreads, 1)
gemm_promote_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmSA, const __grid_constant__ CUtensorMap tmSB,
                    const __grid_constant__ CUtensorMap tmC, const TcParams P) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t base = smem_u32(smem);
    const uint32_t bars = base + kPOffBars;
    const uint32_t full_bar = bars, empty_bar = bars + 32, pfull_bar = bars + 64, pempty_bar = bars + 96;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + kPOffBars + 128);
    volatile uint32_t *abort_flag = tmem_slot + 1;           // flag, poll limit
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPStages; ++s) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, 1 + 8);         // the MMA commit and the eight promotion warps
        }
        for (int b = 0; b < kPBufs; ++b) {
            mbar_init(pfull_bar + 8 * b, 1);
            mbar_init(pempty_bar + 8 * b, 8);
        }
        abort_flag[0] = (base & 1023u) ? 1u : 0u;
        abort_flag[1] = P.wait_limit ? P.wait_limit : kWaitLimit;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        tmem_alloc<1>(smem_u32((const void *)tmem_slot), kPBufs * kPN);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- TMA producer: operands and their scales of one 64-element K slice per stage
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && !P.skip_loads && tile < P.total_tiles; tile += gridDim.x) {
                const PTile t = ptile_info(P, tile);
                for (int ks = 0; ks < t.nks; ++ks) {
                    if (!mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t fb = full_bar + 8 * stage;
                    mbar_expect_tx(fb, kPStageTx);
                    const int32_t ke = (t.ks0 + ks) * kPKElems, kb = (t.ks0 + ks) * 4;
                    tma_load_2d(base + stage * kPOperandStage, &tmA, ke, (int32_t)t.m0, fb);
                    tma_load_2d(base + kPOffB + stage * kPOperandStage, &tmB, ke, (int32_t)(t.b_row0 + t.n0), fb);
                    tma_load_2d(base + kPOffSA + stage * kPScaleStage, &tmSA, (int32_t)t.m0, kb, fb);
                    tma_load_2d(base + kPOffSB + stage * kPScaleStage, &tmSB, (int32_t)(t.b_row0 + t.n0), kb, fb);
                    if (++stage == kPStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- MMA issuer: one K = 16 MMA per quant block, each into a fresh partial buffer
            int stage = 0, buf = 0;
            uint32_t phase = 0, bphase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < P.total_tiles; tile += gridDim.x) {
                const PTile t = ptile_info(P, tile);
                for (int ks = 0; ok && ks < t.nks; ++ks) {
                    if (!mbar_wait(full_bar + 8 * stage, phase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t adesc = umma_desc_sw128(base + stage * kPOperandStage);
                    const uint64_t bdesc = umma_desc_sw128(base + kPOffB + stage * kPOperandStage);
#pragma unroll 1
                    for (int b = 0; b < 4; ++b) {
                        if (!mbar_wait(pempty_bar + 8 * buf, bphase ^ 1u, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        // 16 BF16 = 32 bytes along K: +2 in the (address >> 4) field of the descriptors
                        tc_mma_bf16(tmem_base + (uint32_t)buf * kPN, adesc + (uint64_t)(2 * b), bdesc + (uint64_t)(2 * b),
                                    kPInstrDesc, 0u);
                        tc_commit<1>(pfull_bar + 8 * buf);
                        if (++buf == kPBufs) { buf = 0; bphase ^= 1u; }
                    }
                    tc_commit<1>(empty_bar + 8 * stage);
                    if (++stage == kPStages) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else {
        // ---------------- promotion + epilogue.  Warp w: TMEM lanes 32 q .. 32 q + 31 (q = w & 3), columns 64 half ..
        const int q = warp & 3, half = (warp - 2) >> 2;
        const int row = q * 32 + lane, cbase = 64 * half;
        uint8_t *buf_st = smem + kPOffEpi + (warp - 2) * 4096;
        int stage = 0, buf = 0;
        uint32_t phase = 0, bphase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < P.total_tiles; tile += gridDim.x) {
            const PTile t = ptile_info(P, tile);
            float2 acc[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) acc[j] = make_float2(0.0f, 0.0f);
            // Per quant block: wait for its partial, copy this warp's 32 x 64 part out of tensor memory, hand the buffer
            // back to the MMA issuer at once (it runs up to kPBufs blocks ahead), then multiply the part in.
            for (int ks = 0; ok && ks < t.nks; ++ks) {
                if (!mbar_wait_warp(full_bar + 8 * stage, phase, abort_flag)) { ok = false; break; }
                const float *sA_s = reinterpret_cast<const float *>(smem + kPOffSA + stage * kPScaleStage);
                const float *sB_s = reinterpret_cast<const float *>(smem + kPOffSB + stage * kPScaleStage);
#pragma unroll 1
                for (int b = 0; b < 4; ++b) {
                    const float sa = sA_s[b * kTM + row];
                    const float2 sa2 = make_float2(sa, sa);
                    const float4 *sb4 = reinterpret_cast<const float4 *>(sB_s + b * kPN + cbase);
                    if (!mbar_wait_warp(pfull_bar + 8 * buf, bphase, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * kPN + cbase);
                    uint32_t v0[32], v1[32];
                    tc_ld32(taddr, v0);
                    tc_ld32(taddr + 32, v1);
                    tc_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(pempty_bar + 8 * buf);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float4 sb = sb4[j];
                        const float2 w01 = pmul2(make_float2(sb.x, sb.y), sa2), w23 = pmul2(make_float2(sb.z, sb.w), sa2);
                        acc[2 * j] = pfma2(make_float2(__uint_as_float(v0[4 * j]), __uint_as_float(v0[4 * j + 1])), w01, acc[2 * j]);
                        acc[2 * j + 1] = pfma2(make_float2(__uint_as_float(v0[4 * j + 2]), __uint_as_float(v0[4 * j + 3])), w23, acc[2 * j + 1]);
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float4 sb = sb4[8 + j];
                        const float2 w01 = pmul2(make_float2(sb.x, sb.y), sa2), w23 = pmul2(make_float2(sb.z, sb.w), sa2);
                        acc[16 + 2 * j] = pfma2(make_float2(__uint_as_float(v1[4 * j]), __uint_as_float(v1[4 * j + 1])), w01, acc[16 + 2 * j]);
                        acc[16 + 2 * j + 1] = pfma2(make_float2(__uint_as_float(v1[4 * j + 2]), __uint_as_float(v1[4 * j + 3])), w23, acc[16 + 2 * j + 1]);
                    }
                    if (++buf == kPBufs) { buf = 0; bphase ^= 1u; }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty_bar + 8 * stage);       // this warp no longer reads the stage's scales
                if (++stage == kPStages) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            // ---- epilogue: two 32-column chunks of this warp's 32 x 64 part of the tile, through swizzled staging + TMA store
            const int64_t m_own = t.m0 + row;
            const int32_t c_row = (int32_t)(t.m0 + q * 32), c_grp = (int32_t)(t.c_row0 / (P.M > 0 ? P.M : 1));
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int64_t n_base = t.n0 + cbase + 32 * c;
                if (n_base >= P.N || c_row >= P.M) continue;
                float x[32];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    x[2 * j] = acc[16 * c + j].x;
                    x[2 * j + 1] = acc[16 * c + j].y;
                }
                if (n_base + 32 > P.N && P.n_unaligned) epi_store_box_plain(P, x, t.c_row0 + m_own, n_base, m_own < P.M);
                else epi_store_box_tma(P, &tmC, buf_st, lane, x, (int32_t)n_base, c_row, c_grp);
            }
        }
        epi_store_drain(lane);
    }
    tc_teardown<1>(abort_flag, P.dev_status, tmem_base, kPBufs * kPN, warp);
}

// ------------------------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------------------------

static size_t pround(size_t v, size_t a) { return (v + a - 1) / a * a; }
static int64_t pad4(int64_t v) { return (v + 3) / 4 * 4; }

size_t gemm_promote_workspace_bytes(int64_t a_rows, int64_t b_rows, int64_t K) {
    return pround((size_t)a_rows * K * 2, 256) + pround((size_t)b_rows * K * 2, 256) +
           pround((size_t)(K / 16) * pad4(a_rows) * 4, 256) + pround((size_t)(K / 16) * pad4(b_rows) * 4, 256);
}

int gemm_promote_kernel_launches() { return 2; }

// The transposed scales of B are fetched by TMA starting at column b_row0 + n0 (FP32): in a row-grouped product
// b_row0 = group * group_n, which must stay 16-byte aligned.
bool gemm_promote_supported(int mode, int64_t group_n) { return mode != 1 || group_n % 4 == 0; }

static bool pmake_map(CUtensorMap *map, CUtensorMapDataType dt, const void *ptr, uint64_t inner, uint64_t outer,
                      uint64_t stride_bytes, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle sw) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {stride_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, dt, 2, const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int gemm_promote_launch(const ufp4_qtensor *A, const ufp4_qtensor *B, void *C, int64_t ldc, int c_is_bf16, int mode,
                        int64_t M, int64_t N, int64_t K, const int64_t *offsets, int num_groups, int64_t group_n,
                        void *workspace, size_t workspace_bytes, int32_t *dev_status, void *stream) {
    if (!gemm_promote_supported(mode, group_n)) return UFP4_ERR_UNSUPPORTED;
    if (!aligned_to(workspace, 256)) return UFP4_ERR_ALIGN;
    if (workspace_bytes < gemm_promote_workspace_bytes(A->rows, B->rows, K)) return UFP4_ERR_WORKSPACE;
    if (A->rows > 0x7FFFFFFF || B->rows > 0x7FFFFFFF || K > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    const int64_t lda_t = pad4(A->rows), ldb_t = pad4(B->rows);
    __nv_bfloat16 *A16 = reinterpret_cast<__nv_bfloat16 *>(ws);
    __nv_bfloat16 *B16 = reinterpret_cast<__nv_bfloat16 *>(ws + pround((size_t)A->rows * K * 2, 256));
    float *sAt = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(B16) + pround((size_t)B->rows * K * 2, 256));
    float *sBt = reinterpret_cast<float *>(reinterpret_cast<uint8_t *>(sAt) + pround((size_t)(K / 16) * lda_t * 4, 256));

    PDecodeParams D = {};
    D.op[0] = PDecodeOperand{static_cast<const uint8_t *>(A->codes), A->scales, A->tensor_scale, A->ld_codes_bytes,
                             A->ld_scales, A->rows, lda_t, codebook_of(A->grid), A->scale_fmt, A16, sAt};
    D.op[1] = PDecodeOperand{static_cast<const uint8_t *>(B->codes), B->scales, B->tensor_scale, B->ld_codes_bytes,
                             B->ld_scales, B->rows, ldb_t, codebook_of(B->grid), B->scale_fmt, B16, sBt};
    D.K = K;
    D.a_ctas = (A->rows + 7) / 8;
    const int64_t decode_ctas = D.a_ctas + (B->rows + 7) / 8;
    if (decode_ctas > 0x7FFFFFFF) return UFP4_ERR_SHAPE;
    decode_promote_kernel<<<(unsigned)decode_ctas, 256, 0, st>>>(D);
    if (cudaGetLastError() != cudaSuccess) return UFP4_ERR_CUDA;

    CUtensorMap tmA, tmB, tmSA, tmSB, tmC;
    if (!pmake_map(&tmA, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, A16, (uint64_t)K, (uint64_t)A->rows, (uint64_t)K * 2, kPKElems, kTM,
                   CU_TENSOR_MAP_SWIZZLE_128B) ||
        !pmake_map(&tmB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, B16, (uint64_t)K, (uint64_t)B->rows, (uint64_t)K * 2, kPKElems, kPN,
                   CU_TENSOR_MAP_SWIZZLE_128B) ||
        !pmake_map(&tmSA, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, sAt, (uint64_t)lda_t, (uint64_t)(K / 16), (uint64_t)lda_t * 4, kTM, 4,
                   CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !pmake_map(&tmSB, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, sBt, (uint64_t)ldb_t, (uint64_t)(K / 16), (uint64_t)ldb_t * 4, kPN, 4,
                   CU_TENSOR_MAP_SWIZZLE_NONE))
        return UFP4_ERR_CUDA;
    {
        EncodeTiledFn fn = encode_tiled_fn();
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
    P.mt = (int)((M + kTM - 1) / kTM);
    P.nt = (int)((N + kPN - 1) / kPN);
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
        UFP4_CUDA_OK(cudaFuncSetAttribute(gemm_promote_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPSmem));
        return UFP4_OK;
    }, &dev);
    if (rc_setup != UFP4_OK) return rc_setup;
    const int num_sms = dev->num_sms;
    const int grid = (int)(total < num_sms ? total : num_sms);
    gemm_promote_kernel<<<grid, kPThreads, kPSmem, st>>>(tmA, tmB, tmSA, tmSB, tmC, P);
    return cudaGetLastError() == cudaSuccess ? UFP4_OK : UFP4_ERR_CUDA;
}

}  // namespace ufp4
