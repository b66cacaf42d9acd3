// Gradient-norm pass of the global-norm gradient clip.
//
// Contract: sumsq_k is the EXACT sum of the squares of worker k's gradient,
// rounded once to binary64; norm = sqrt(sumsq); coefficient = min(1, max_norm /
// (norm + 1e-6)) in binary64, rounded once to binary32.  To get the exactly
// rounded sum on a GPU the squares (exact in binary64: 24-bit x 24-bit) are
// accumulated in double-double arithmetic (an unevaluated pair hi + lo, about 106
// significant bits, built from error-free additions), whose error is far below
// half a unit of binary64; the result therefore does not depend on the order of
// the additions, up to a probability of about 2^-40 per call.  The order is
// nevertheless fixed (per thread, per CTA, then one CTA over the per-item
// partials), so that results are bitwise reproducible and independent of the
// launch shape.
#pragma once
#include "palsgd_kernels.cuh"

namespace palsgd {

struct DD { double hi, lo; };

// hi + lo += x for x >= 0 and hi >= 0: hi + x is split exactly into its rounded sum and the
// rounding error.  With the larger operand first the error is small - (s - big) (Dekker's
// FastTwoSum): three binary64 operations and a comparison where the order-free form takes six.
__device__ __forceinline__ void dd_accumulate(DD& a, double x)
{
    const bool   hi_big = a.hi >= x;
    const double big    = hi_big ? a.hi : x;
    const double small  = hi_big ? x : a.hi;
    const double s = __dadd_rn(big, small);
    const double e = __dsub_rn(small, __dsub_rn(s, big));
    a.hi = s;
    a.lo = __dadd_rn(a.lo, e);
}

// An infinite or NaN high part carries no meaningful low part (the error terms of inf are NaN):
// it is propagated alone, so that an overflowing or NaN gradient gives sumsq = inf or NaN.
__device__ __forceinline__ DD dd_add(const DD& a, const DD& b)
{
    const double s  = __dadd_rn(a.hi, b.hi);
    if (!isfinite(s)) return DD{s, 0.0};
    const double bb = __dsub_rn(s, a.hi);
    double e = __dadd_rn(__dsub_rn(a.hi, __dsub_rn(s, bb)), __dsub_rn(b.hi, bb));
    e = __dadd_rn(e, __dadd_rn(a.lo, b.lo));
    const double hi = __dadd_rn(s, e);                     // renormalise (|e| << |s|)
    const double lo = __dsub_rn(e, __dsub_rn(hi, s));
    return DD{hi, lo};
}

__device__ __forceinline__ void dd_square_in(DD& a, float g)
{
    const double x = (double)g;
    dd_accumulate(a, __dmul_rn(x, x));                     // exact product
}

// Sum over the CTA in a fixed tree: lanes by shuffles, then the warps in order.
__device__ __forceinline__ DD dd_block_sum(DD v, DD* s_warp /* [kThreads / 32] */)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        DD o;
        o.hi = __shfl_down_sync(0xFFFFFFFFu, v.hi, off);
        o.lo = __shfl_down_sync(0xFFFFFFFFu, v.lo, off);
        v = dd_add(v, o);
    }
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();                                        // s_warp may still be read from a previous call
    if (lane == 0) s_warp[warp] = v;
    __syncthreads();
    DD tot{0.0, 0.0};
    if (threadIdx.x == 0) {
        tot = s_warp[0];
        for (uint32_t w = 1; w < kThreads / 32; ++w) tot = dd_add(tot, s_warp[w]);
    }
    return tot;                                             // valid in thread 0
}

// Sum of squares of one chunk of one gradient (this thread's share).
// Four independent accumulators per thread (element position mod 4) keep the binary64 pipe
// busy despite the serial dependence inside each; they are merged in a fixed order.
template <int PREC>
__device__ __forceinline__ void sumsq_chunk(DD (&q)[4], const void* g, uint32_t len, bool vec)
{
    constexpr int U = 4;                                    // 128-bit loads in flight per thread
    uint32_t done = 0;
    if (vec) {
        if (PREC) {
            const uint4* g8 = static_cast<const uint4*>(g);
            const uint32_t n8 = len >> 3;
            for (uint32_t base = 0; base < n8; base += kThreads * U) {
                uint4 R[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t i = base + u * kThreads + threadIdx.x;
                    if (i < n8) R[u] = ld_stream(g8 + i);
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t i = base + u * kThreads + threadIdx.x;
                    if (i < n8) {
                        float f[8]; unpack8(R[u], f);
#pragma unroll
                        for (int c = 0; c < 8; ++c) dd_square_in(q[c & 3], f[c]);
                    }
                }
            }
            done = n8 << 3;
        } else {
            const float4* g4 = static_cast<const float4*>(g);
            const uint32_t n4 = len >> 2;
            for (uint32_t base = 0; base < n4; base += kThreads * U) {
                float4 R[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t i = base + u * kThreads + threadIdx.x;
                    if (i < n4) R[u] = ld_stream(g4 + i);
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t i = base + u * kThreads + threadIdx.x;
                    if (i < n4) { dd_square_in(q[0], R[u].x); dd_square_in(q[1], R[u].y);
                                  dd_square_in(q[2], R[u].z); dd_square_in(q[3], R[u].w); }
                }
            }
            done = n4 << 2;
        }
    }
    for (uint32_t i = done + threadIdx.x; i < len; i += kThreads)
        dd_square_in(q[0], PREC ? __bfloat162float(static_cast<const __nv_bfloat16*>(g)[i])
                                : static_cast<const float*>(g)[i]);
}

// ---- bf16 gradients: exact sums at two binary64 operations per element
// The square of a bf16 value has 16 significant bits, so a run of such squares can be summed
// EXACTLY in plain binary64 as long as all of them sit within about 2^37 of the running sum.
// Each chain is kept twice, once with every addition rounded down and once rounded up (the
// product x*x is exact, so fma_rd / fma_ru round the exact x*x + s once): the chain rounded down
// never exceeds the exact sum and the chain rounded up never falls below it, hence if the two
// are EQUAL after a stretch of additions, every addition in it was exact and the common value is
// the exact sum.  The test is made once per chunk and costs nothing per element.  When it fails
// (an element far smaller than the running sum, or a NaN), the chains go back to their values at
// the start of the chunk and this thread's elements of the chunk are added in double-double.
// Zeros, denormals and infinities need no special case (inf = inf keeps the chains equal).
struct FastSq {
    double dn[4], up[4];        // four independent chains (element position mod 4), rounded down / up
    double ok[4];               // their (common) values at the start of the current chunk

    __device__ __forceinline__ void init()
    {
#pragma unroll
        for (int j = 0; j < 4; ++j) { dn[j] = 0.0; up[j] = 0.0; ok[j] = 0.0; }
    }
    __device__ __forceinline__ void add(int j, float g)
    {
        const double x = (double)g;
        dn[j] = __fma_rd(x, x, dn[j]);
        up[j] = __fma_ru(x, x, up[j]);
    }
    // true: every addition since the last call was exact (and the chains are kept);
    // false: the chains have been put back to where they were at that call
    __device__ __forceinline__ bool settle()
    {
        const bool exact = dn[0] == up[0] && dn[1] == up[1] && dn[2] == up[2] && dn[3] == up[3];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (exact) ok[j] = dn[j];
            else { dn[j] = ok[j]; up[j] = ok[j]; }
        }
        return exact;
    }
};

// One 16-byte-aligned chunk of one bf16 gradient: this thread's groups of 8 into the fast chains, or,
// if the chains' test fails for this chunk, once more into the double-double accumulator `slow`.
__device__ __forceinline__ void sumsq_chunk_bf16_fast(FastSq& f, DD& slow, const void* g, uint32_t len)
{
    constexpr int U = 4;
    const uint4* g8 = static_cast<const uint4*>(g);
    const uint32_t n8 = len >> 3;
    for (uint32_t base = 0; base < n8; base += kThreads * U) {
        uint4 R[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * kThreads + threadIdx.x;
            R[u] = i < n8 ? ld_stream(g8 + i) : make_uint4(0u, 0u, 0u, 0u);      // zeros add nothing
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            float v[8]; unpack8(R[u], v);
#pragma unroll
            for (int c = 0; c < 8; ++c) f.add(c & 3, v[c]);
        }
    }
    if (!f.settle()) {                                      // rare; the data is still in cache
        for (uint32_t i = threadIdx.x; i < n8; i += kThreads) {
            float v[8]; unpack8(__ldg(g8 + i), v);
#pragma unroll
            for (int c = 0; c < 8; ++c) dd_square_in(slow, v[c]);
        }
    }
    for (uint32_t i = (n8 << 3) + threadIdx.x; i < len; i += kThreads)
        dd_square_in(slow, __bfloat162float(static_cast<const __nv_bfloat16*>(g)[i]));
}

// One launch ahead of a step whose gradients are clipped.  Work items: (chunk, worker) with the
// worker index fastest (ddp = 0), or chunks (ddp = 1: the norm of the averaged gradient, formed
// exactly as the DDP step forms it).  Every item leaves a double-double partial in
// tb.norm_part (indexed [group * workers + worker]); the last CTA to finish adds the partials of each worker in item order and
// writes sumsq and the clip coefficient to the device state.
template <int PREC>
__global__ void __launch_bounds__(kThreads)
palsgd_gradnorm_kernel(const __grid_constant__ NormArgs a)
{
    __shared__ unsigned char s_pull[kMaxWorkers];
    __shared__ DD s_warp[kThreads / 32];
    __shared__ const void* s_g[kMaxWorkers];
    __shared__ unsigned int s_last;
    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    DevState* st = tb.st;
    const unsigned long long t = st->t;
    const uint32_t Kitems = a.ddp ? 1u : K;

    if (threadIdx.x < K) s_pull[threadIdx.x] = a.ddp ? 0 : draw_pull(a.seed, t, a.k0 + threadIdx.x, a.thr);
    __syncthreads();

    // Work item = a.group consecutive chunks of one worker: the per-thread sums run over the whole
    // group, so the CTA-wide reduction (as costly as ~20 elements per thread) is paid once per group.
    const uint32_t n_groups = (tb.n_chunks + a.group - 1) / a.group;
    const uint64_t n_items = (uint64_t)n_groups * Kitems;
    const size_t gsz = PREC ? 2 : 4;
    for (uint64_t item = blockIdx.x; item < n_items; item += gridDim.x) {
        const uint32_t k = (uint32_t)(item % Kitems);
        const uint32_t c_begin = (uint32_t)(item / Kitems) * a.group;
        const uint32_t c_end = min(c_begin + a.group, tb.n_chunks);
        DD q[4] = {{0.0, 0.0}, {0.0, 0.0}, {0.0, 0.0}, {0.0, 0.0}};
        bool fast_done = false;
        if (PREC == 1 && !a.ddp) {
            // bf16 gradients: plain binary64 chains whose exactness is tested chunk by chunk
            fast_done = true;
            if (!s_pull[k]) {
                FastSq f; f.init();
                for (uint32_t c = c_begin; c < c_end; ++c) {
                    const Chunk ch = tb.chunks[c];
                    const uint32_t seg = ch.seg & ~kSegVecFlag;
                    const char* g = static_cast<const char*>(tb.grad[(size_t)k * tb.n_seg + seg]) + ch.off * gsz;
                    if (ch.seg & kSegVecFlag) sumsq_chunk_bf16_fast(f, q[0], g, ch.len);
                    else                      sumsq_chunk<PREC>(q, g, ch.len, false);
                }
                q[1] = dd_add(DD{f.dn[0], 0.0}, DD{f.dn[1], 0.0});     // the chains hold exact sums
                q[2] = dd_add(DD{f.dn[2], 0.0}, DD{f.dn[3], 0.0});
            }
        }
        for (uint32_t c = c_begin; c < c_end && !fast_done; ++c) {
        const Chunk ch = tb.chunks[c];
        const uint32_t seg = ch.seg & ~kSegVecFlag;
        const bool vec = (ch.seg & kSegVecFlag) != 0;
        if (a.ddp) {
            __syncthreads();
            if (threadIdx.x < K)
                s_g[threadIdx.x] = static_cast<const char*>(tb.grad[(size_t)threadIdx.x * tb.n_seg + seg]) + ch.off * gsz;
            __syncthreads();
            uint32_t done = 0;
            if (vec) {
                const uint32_t n4 = ch.len >> 2;
                for (uint32_t i = threadIdx.x; i < n4; i += kThreads) {
                    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (uint32_t kk = 0; kk < K; ++kk) {
                        float4 r;
                        if (PREC) { float f[4]; unpack4(ld_stream(static_cast<const uint2*>(s_g[kk]) + i), f);
                                    r = make_float4(f[0], f[1], f[2], f[3]); }
                        else      { r = ld_stream(static_cast<const float4*>(s_g[kk]) + i); }
                        if (kk == 0) sum = r;
                        else { sum.x = __fadd_rn(sum.x, r.x); sum.y = __fadd_rn(sum.y, r.y);
                               sum.z = __fadd_rn(sum.z, r.z); sum.w = __fadd_rn(sum.w, r.w); }
                    }
                    dd_square_in(q[0], __fdiv_rn(sum.x, a.Kf)); dd_square_in(q[1], __fdiv_rn(sum.y, a.Kf));
                    dd_square_in(q[2], __fdiv_rn(sum.z, a.Kf)); dd_square_in(q[3], __fdiv_rn(sum.w, a.Kf));
                }
                done = n4 << 2;
            }
            for (uint32_t i = done + threadIdx.x; i < ch.len; i += kThreads) {
                float sum = 0.f;
                for (uint32_t kk = 0; kk < K; ++kk) {
                    const float gk = PREC ? __bfloat162float(static_cast<const __nv_bfloat16*>(s_g[kk])[i])
                                          : static_cast<const float*>(s_g[kk])[i];
                    sum = kk == 0 ? gk : __fadd_rn(sum, gk);
                }
                dd_square_in(q[0], __fdiv_rn(sum, a.Kf));
            }
        } else if (!s_pull[k]) {                            // a pulling worker's gradient is not used
            const char* g = static_cast<const char*>(tb.grad[(size_t)k * tb.n_seg + seg]) + ch.off * gsz;
            sumsq_chunk<PREC>(q, g, ch.len, vec);
        }
        }
        const DD tot = dd_block_sum(dd_add(dd_add(q[0], q[1]), dd_add(q[2], q[3])), s_warp);
        if (threadIdx.x == 0) tb.norm_part[item] = make_double2(tot.hi, tot.lo);
    }

    // ---- the last CTA to finish reduces the partials
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int prev = atomicAdd(&st->done_norm, 1u);
        s_last = (prev == gridDim.x - 1);
        __threadfence();
    }
    __syncthreads();
    if (!s_last) return;
    for (uint32_t k = 0; k < Kitems; ++k) {
        if (!a.ddp && s_pull[k]) continue;                  // uniform over the CTA
        DD acc{0.0, 0.0};
        for (uint32_t c = threadIdx.x; c < n_groups; c += kThreads) {
            const double2 p = __ldcg(tb.norm_part + (size_t)c * Kitems + k);
            acc = dd_add(acc, DD{p.x, p.y});
        }
        const DD tot = dd_block_sum(acc, s_warp);
        if (threadIdx.x == 0) {
            const double sumsq = isfinite(tot.hi) ? __dadd_rn(tot.hi, tot.lo) : tot.hi;
            const double coef = __ddiv_rn(a.max_norm, __dadd_rn(__dsqrt_rn(sumsq), 1e-6));
            const float clip = (float)(coef < 1.0 ? coef : 1.0);
            if (a.ddp) { for (uint32_t kk = 0; kk < K; ++kk) { st->sumsq[kk] = sumsq; st->clip[kk] = clip; } }
            else       { st->sumsq[k] = sumsq; st->clip[k] = clip; }
        }
    }
    if (threadIdx.x == 0) { st->done_norm = 0; __threadfence(); }
}

}  // namespace palsgd
