// Philox4x32-10 counter-based generator (Salmon et al., SC'11) and the branch
// draw of Algorithm 1 built on it.  Host and device share this header so the
// host-side palsgd_decision() and the kernels cannot drift apart.
#pragma once
#include <stdint.h>

namespace palsgd {

struct U32x4 { uint32_t a, b, c, d; };

__host__ __device__ __forceinline__ uint32_t mul_hi32(uint32_t x, uint32_t y)
{
#ifdef __CUDA_ARCH__
    return __umulhi(x, y);
#else
    return (uint32_t)(((uint64_t)x * (uint64_t)y) >> 32);
#endif
}

// counter (a,b,c,d), key (k0,k1) -> four 32-bit words after ten rounds
__host__ __device__ __forceinline__ U32x4 philox4x32_10(U32x4 ctr, uint32_t k0, uint32_t k1)
{
    constexpr uint32_t kMulA = 0xD2511F53u, kMulB = 0xCD9E8D57u;
    constexpr uint32_t kWeyl0 = 0x9E3779B9u, kWeyl1 = 0xBB67AE85u;
#ifdef __CUDA_ARCH__
#pragma unroll
#endif
    for (int r = 0; r < 10; ++r) {
        const uint32_t hiA = mul_hi32(kMulA, ctr.a), loA = kMulA * ctr.a;
        const uint32_t hiB = mul_hi32(kMulB, ctr.c), loB = kMulB * ctr.c;
        ctr = U32x4{hiB ^ ctr.b ^ k0, loB, hiA ^ ctr.d ^ k1, loA};
        k0 += kWeyl0;
        k1 += kWeyl1;
    }
    return ctr;
}

// Algorithm 1's branch draw (a uniform variate compared with p).  One draw per (worker k, step t):
// word 0 of Philox with counter (t_lo, t_hi, k, 0) and key (seed_lo, seed_hi),
// compared with thr = floor(p * 2^32).
__host__ __device__ __forceinline__ bool draw_pull(uint64_t seed, uint64_t t, uint32_t k, uint64_t thr)
{
    const U32x4 w = philox4x32_10(U32x4{(uint32_t)t, (uint32_t)(t >> 32), k, 0u},
                                  (uint32_t)seed, (uint32_t)(seed >> 32));
    return (uint64_t)w.a < thr;
}

}  // namespace palsgd
