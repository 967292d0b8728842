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
