// Shared device/host helpers of libufp4 (CUDA side only; the CPU oracle shares none of this).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ufp4.h"

namespace ufp4 {

// ---------------------------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): the counter-based generator behind the RHT signs and the SR random bytes.
// ---------------------------------------------------------------------------------------------------------------
struct Philox4 {
    uint32_t x, y, z, w;
};

__host__ __device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                          uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
#ifdef __CUDA_ARCH__
        uint32_t lo0 = 0xD2511F53u * c0, hi0 = __umulhi(0xD2511F53u, c0);
        uint32_t lo1 = 0xCD9E8D57u * c2, hi1 = __umulhi(0xCD9E8D57u, c2);
#else
        uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t lo0 = (uint32_t)p0, hi0 = (uint32_t)(p0 >> 32), lo1 = (uint32_t)p1, hi1 = (uint32_t)(p1 >> 32);
#endif
        uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return Philox4{c0, c1, c2, c3};
}

constexpr uint32_t kRhtCounterTag = 0x52485400u;  // counter word 3 of the sign draw
constexpr uint32_t kSrCounterTag = 0x53520000u;   // counter word 3 of the SR draws

// The codebook behind a tensor's nibbles: the range-restricted E2M1 grids store plain E2M1 codes.
inline int codebook_of(int grid) { return grid > UFP4_GRID_E2M1 ? (int)UFP4_GRID_E2M1 : grid; }

// Scale formats whose stored scales are FP32 powers of two.
inline bool is_pow2_fmt(int scale_fmt) { return scale_fmt == UFP4_SCALE_POW2 || scale_fmt == UFP4_SCALE_E8M0_B32; }

inline bool aligned_to(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

#define UFP4_CUDA_OK(expr)                                \
    do {                                                  \
        cudaError_t e_ = (expr);                          \
        if (e_ != cudaSuccess) return UFP4_ERR_CUDA;      \
    } while (0)

}  // namespace ufp4
