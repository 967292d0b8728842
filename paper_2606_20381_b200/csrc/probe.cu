// Issue-rate probe (a measurement aid, not on the hot path; the paper has no counterpart): how many cycles a scheduler
// needs per warp instruction for the instruction kinds the quantizer is made of, alone and in pairs.  One CTA of 1024
// threads per SM (8 warps per scheduler), eight independent chains per thread, clock64 around the loop.
#include "common.cuh"

namespace ufp4 {

#define UFP4_P_F2(d, c) asm volatile("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%0, %1}; mov.b64 rb, {%2, %3}; add.rn.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd; }" : "+f"(d.x), "+f"(d.y) : "f"(c.x), "f"(c.y))
#define UFP4_P_FADD(x, c) asm volatile("add.rn.f32 %0, %0, %1;" : "+f"(x) : "f"(c))
#define UFP4_P_LOP(x, m) asm volatile("lop3.b32 %0, %0, %1, %1, 0x96;" : "+r"(x) : "r"(m))
#define UFP4_P_IMAD(x, m) asm volatile("mad.lo.u32 %0, %0, %1, %1;" : "+r"(x) : "r"(m))

constexpr int kProbeModes = 8;

template <int MODE>
__global__ void __launch_bounds__(1024, 1) probe_kernel(float *sink, long long *cycles, int iters) {
    extern __shared__ char one_cta_per_sm[];
    float2 f[8];
    unsigned u[8];
    for (int i = 0; i < 8; ++i) {
        f[i] = make_float2(threadIdx.x * 0.001f + i, i * 0.5f);
        u[i] = threadIdx.x * 7 + i;
    }
    const float2 c = make_float2(1.0001f, 0.9999f);
    const unsigned m = 0x0F0F0F0Fu + threadIdx.x;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (MODE == 0) UFP4_P_F2(f[i], c);
                if (MODE == 1) { UFP4_P_FADD(f[i].x, c.x); UFP4_P_FADD(f[i].y, c.y); }
                if (MODE == 2) UFP4_P_LOP(u[i], m);
                if (MODE == 3) UFP4_P_IMAD(u[i], m);
                if (MODE == 4) { UFP4_P_F2(f[i], c); UFP4_P_LOP(u[i], m); }
                if (MODE == 5) { UFP4_P_F2(f[i], c); UFP4_P_IMAD(u[i], m); }
                if (MODE == 6) { UFP4_P_F2(f[i], c); UFP4_P_LOP(u[i], m); UFP4_P_LOP(u[(i + 4) & 7], m); }
                if (MODE == 7) { UFP4_P_FADD(f[i].x, c.x); UFP4_P_FADD(f[i].y, c.y); UFP4_P_LOP(u[i], m); }
            }
        }
    }
    __syncthreads();
    const long long t1 = clock64();
    float s = 0.0f;
    unsigned su = 0u;
    for (int i = 0; i < 8; ++i) {
        s += f[i].x + f[i].y;
        su ^= u[i];
    }
    sink[blockIdx.x * blockDim.x + threadIdx.x] = s + (float)su;
    if (threadIdx.x == 0 && blockIdx.x == 0) *cycles = t1 - t0;
}

template <int MODE>
static int run_mode(float *sink, long long *dev_cycles, int num_sms, int iters, cudaStream_t st, double *out) {
    constexpr int kSmem = 200 * 1024;                           // forces one CTA per SM
    UFP4_CUDA_OK(cudaFuncSetAttribute(probe_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem));
    for (int rep = 0; rep < 2; ++rep) probe_kernel<MODE><<<num_sms, 1024, kSmem, st>>>(sink, dev_cycles, iters);
    long long h = 0;
    UFP4_CUDA_OK(cudaMemcpyAsync(&h, dev_cycles, sizeof(h), cudaMemcpyDeviceToHost, st));
    UFP4_CUDA_OK(cudaStreamSynchronize(st));
    *out = (double)h / ((double)iters * 32.0 * 8.0);            // cycles per group of instructions, 8 warps per scheduler
    return UFP4_OK;
}

// ------------------------------------------------------------------------------------------------------------------
// Decode-rate probe: how fast one SM turns a pipeline stage of packed nibbles (a CTA pair's share of a 256 x 256 x 128 step:
// 128 rows of A and 128 rows of B, 128 elements each) into the 128B-swizzled E5M2 operand tiles a tcgen05 MMA reads, all in
// shared memory, with the arithmetic of the folded path's decode pass (16-entry table in four registers, the block's
// exponent offset added to the table, three byte permutes per four nibbles).  THREADS threads share the stage's 2048
// sixteen-element blocks; the result is cycles per stage.
// ------------------------------------------------------------------------------------------------------------------
template <int THREADS>
__global__ void __launch_bounds__(THREADS, 1) probe_decode_kernel(uint32_t *sink, long long *cycles, int iters) {
    extern __shared__ __align__(1024) uint8_t dsm[];
    uint8_t *nib = dsm;                         // [256 rows][64 bytes]
    uint8_t *dexp = dsm + 16384;                // [256 rows][8 blocks] exponent offsets
    uint8_t *out = dsm + 32768;                 // [256 rows][128 bytes], 16-byte piece c of row r at piece c ^ (r & 7)
    for (int i = threadIdx.x; i < 16384 / 4; i += THREADS) reinterpret_cast<uint32_t *>(nib)[i] = 0x9E3779B9u * (uint32_t)(i + 1);
    for (int i = threadIdx.x; i < 2048; i += THREADS) dexp[i] = (uint8_t)(i % 13);
    __syncthreads();
    const uint32_t lutp_lo0 = 0x42403C00u, lutp_hi0 = 0x47464544u, lutn_lo0 = 0xC5C6C7C8u, lutn_hi0 = 0xBCC0C2C4u;
    uint32_t acc = 0u;
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll 4
        for (int item = threadIdx.x; item < 2048; item += THREADS) {
            const int row = item >> 3, blk = item & 7;
            const uint2 cw = *reinterpret_cast<const uint2 *>(nib + row * 64 + blk * 8);
            const uint32_t d = dexp[item] + (uint32_t)(it & 1);
            const uint32_t lutp_lo = lutp_lo0 + d * 0x04040400u, lutp_hi = lutp_hi0 + d * 0x04040404u;
            const uint32_t lutn_lo = lutn_lo0 + d * 0x04040404u, lutn_hi = lutn_hi0 + d * 0x04040404u;
            uint32_t o[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t w = (q & 2 ? cw.y : cw.x) >> (q & 1 ? 16 : 0);
                const uint32_t sel = w & 0x7777u;
                const uint32_t pos = __byte_perm(lutp_lo, lutp_hi, sel), neg = __byte_perm(lutn_lo, lutn_hi, sel);
                o[q] = __byte_perm(pos, neg, ((w >> 1) & 0x4444u) | 0x3210u);
            }
            *reinterpret_cast<uint4 *>(out + row * 128 + ((blk ^ (row & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
        }
        __syncthreads();                        // a stage is handed over as a whole
        acc += out[(threadIdx.x * 16 + it) & 32767];
    }
    const long long t1 = clock64();
    sink[blockIdx.x * THREADS + threadIdx.x] = acc;
    if (threadIdx.x == 0 && blockIdx.x == 0) *cycles = t1 - t0;
}

template <int THREADS>
static int run_decode(uint32_t *sink, long long *dev_cycles, int num_sms, int iters, cudaStream_t st, double *out) {
    constexpr int kSmem = 200 * 1024;                           // forces one CTA per SM
    UFP4_CUDA_OK(cudaFuncSetAttribute(probe_decode_kernel<THREADS>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem));
    for (int rep = 0; rep < 2; ++rep) probe_decode_kernel<THREADS><<<num_sms, THREADS, kSmem, st>>>(sink, dev_cycles, iters);
    long long h = 0;
    UFP4_CUDA_OK(cudaMemcpyAsync(&h, dev_cycles, sizeof(h), cudaMemcpyDeviceToHost, st));
    UFP4_CUDA_OK(cudaStreamSynchronize(st));
    *out = (double)h / (double)iters;                           // cycles per stage of 32768 elements
    return UFP4_OK;
}

}  // namespace ufp4

extern "C" int ufp4_probe_issue_rates(void *dev_scratch, size_t scratch_bytes, double *host_cycles, void *stream) {
    using namespace ufp4;
    if (!dev_scratch || !host_cycles) return UFP4_ERR_NULL;
    int dev = 0, num_sms = 0;
    UFP4_CUDA_OK(cudaGetDevice(&dev));
    UFP4_CUDA_OK(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
    if (scratch_bytes < (size_t)num_sms * 1024 * sizeof(float) + 256) return UFP4_ERR_WORKSPACE;
    if (!aligned_to(dev_scratch, 256)) return UFP4_ERR_ALIGN;
    long long *cyc = static_cast<long long *>(dev_scratch);
    float *sink = reinterpret_cast<float *>(static_cast<uint8_t *>(dev_scratch) + 256);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int iters = 2000;
    int rc;
    if ((rc = run_mode<0>(sink, cyc, num_sms, iters, st, host_cycles + 0)) != UFP4_OK) return rc;
    if ((rc = run_mode<1>(sink, cyc, num_sms, iters, st, host_cycles + 1)) != UFP4_OK) return rc;
    if ((rc = run_mode<2>(sink, cyc, num_sms, iters, st, host_cycles + 2)) != UFP4_OK) return rc;
    if ((rc = run_mode<3>(sink, cyc, num_sms, iters, st, host_cycles + 3)) != UFP4_OK) return rc;
    if ((rc = run_mode<4>(sink, cyc, num_sms, iters, st, host_cycles + 4)) != UFP4_OK) return rc;
    if ((rc = run_mode<5>(sink, cyc, num_sms, iters, st, host_cycles + 5)) != UFP4_OK) return rc;
    if ((rc = run_mode<6>(sink, cyc, num_sms, iters, st, host_cycles + 6)) != UFP4_OK) return rc;
    return run_mode<7>(sink, cyc, num_sms, iters, st, host_cycles + 7);
}

extern "C" int ufp4_probe_decode_rate(void *dev_scratch, size_t scratch_bytes, double *host_cycles, void *stream) {
    using namespace ufp4;
    if (!dev_scratch || !host_cycles) return UFP4_ERR_NULL;
    int dev = 0, num_sms = 0;
    UFP4_CUDA_OK(cudaGetDevice(&dev));
    UFP4_CUDA_OK(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev));
    if (scratch_bytes < (size_t)num_sms * 1024 * sizeof(uint32_t) + 256) return UFP4_ERR_WORKSPACE;
    if (!aligned_to(dev_scratch, 256)) return UFP4_ERR_ALIGN;
    long long *cyc = static_cast<long long *>(dev_scratch);
    uint32_t *sink = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(dev_scratch) + 256);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int iters = 500;
    int rc;
    if ((rc = run_decode<128>(sink, cyc, num_sms, iters, st, host_cycles + 0)) != UFP4_OK) return rc;
    if ((rc = run_decode<256>(sink, cyc, num_sms, iters, st, host_cycles + 1)) != UFP4_OK) return rc;
    if ((rc = run_decode<512>(sink, cyc, num_sms, iters, st, host_cycles + 2)) != UFP4_OK) return rc;
    return run_decode<1024>(sink, cyc, num_sms, iters, st, host_cycles + 3);
}
