// PALSGD kernels for sm_100a: fused inner step (branch draw + AdamW / momentum
// SGD / pull), forced pull, outer sync (K-way average + Nesterov + broadcast),
// and set-up.  All of them are HBM-bandwidth-bound streaming kernels: 128-bit
// coalesced accesses, enough independent loads in flight per thread to cover
// DRAM latency, streaming cache hints on data that is touched once per launch.
//
// Every element operation is written with the round-to-nearest intrinsics
// (__fmul_rn, __fadd_rn, ...): they are single IEEE binary32 operations that
// the compiler never fuses into a multiply-add, whatever flags are in force.
#pragma once
#include "palsgd_device.cuh"
#include "palsgd_philox.cuh"

namespace palsgd {

// ---------------------------------------------------------------- element math

// clip: the global-norm clip coefficient the gradient is multiplied by first (1 = no clipping;
// the multiplication by 1 is exact, so one code path serves both cases).
struct AdamScalars { float b1, b2, omb1, omb2, bc1, bc2, decay, lr, eps; float clip = 1.f; };
struct SgdScalars  { float mu, wd, lr; float clip = 1.f; };

// AdamW with decoupled decay and bias correction (gradient branch, Eq. (1)).
__device__ __forceinline__ void adamw_elem(float g, float& x, float& m, float& v, const AdamScalars& s)
{
    g = __fmul_rn(g, s.clip);
    m = __fadd_rn(__fmul_rn(s.b1, m), __fmul_rn(s.omb1, g));
    v = __fadd_rn(__fmul_rn(s.b2, v), __fmul_rn(s.omb2, __fmul_rn(g, g)));
    const float mh = __fdiv_rn(m, s.bc1);
    const float vh = __fdiv_rn(v, s.bc2);
    x = __fmul_rn(x, s.decay);
    x = __fsub_rn(x, __fmul_rn(s.lr, __fdiv_rn(mh, __fadd_rn(__fsqrt_rn(vh), s.eps))));
}

// Momentum SGD, L2 decay folded into the gradient (gradient branch, Eq. (1)).
__device__ __forceinline__ void sgdm_elem(float g, float& x, float& buf, const SgdScalars& s)
{
    g = __fmul_rn(g, s.clip);
    const float gp = __fadd_rn(g, __fmul_rn(s.wd, x));
    buf = __fadd_rn(__fmul_rn(s.mu, buf), gp);
    x = __fsub_rn(x, __fmul_rn(s.lr, buf));
}

// Pseudo-synchronisation (Eq. (2)): x <- x - beta (x - x_g).
__device__ __forceinline__ float pull_elem(float x, float xg, float beta)
{
    return __fsub_rn(x, __fmul_rn(beta, __fsub_rn(x, xg)));
}

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t h16) { return __uint_as_float(h16 << 16); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);      // RNE, .x in the low half
    return *reinterpret_cast<const uint32_t*>(&v);
}

// streaming (touched once per launch) 128-bit accesses
__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }
__device__ __forceinline__ uint4  ld_stream(const uint4* p)  { return __ldcs(p); }
__device__ __forceinline__ uint2  ld_stream(const uint2* p)  { return __ldcs(p); }
__device__ __forceinline__ void   st_stream(float4* p, float4 v) { __stcs(p, v); }
__device__ __forceinline__ void   st_stream(uint4* p, uint4 v)   { __stcs(p, v); }
__device__ __forceinline__ void   st_stream(uint2* p, uint2 v)   { __stcs(p, v); }

#define PALSGD_FOR4(EXPR)  { constexpr int c = 0; EXPR; } { constexpr int c = 1; EXPR; } \
                           { constexpr int c = 2; EXPR; } { constexpr int c = 3; EXPR; }
__device__ __forceinline__ float& comp(float4& a, int c) { return c == 0 ? a.x : c == 1 ? a.y : c == 2 ? a.z : a.w; }
__device__ __forceinline__ float  compv(const float4& a, int c) { return c == 0 ? a.x : c == 1 ? a.y : c == 2 ? a.z : a.w; }

// ---------------------------------------------------------------- fp32 chunk bodies

// U independent 128-bit loads per stream are issued before any arithmetic.
template <int U, int NT>
__device__ __forceinline__ void adamw_chunk_f32(uint32_t tid, const float* __restrict__ g, float* __restrict__ x,
                                                float* __restrict__ m, float* __restrict__ v,
                                                uint32_t len, const AdamScalars& s)
{
    const uint32_t n4 = len >> 2;
    const float4* g4 = reinterpret_cast<const float4*>(g);
    float4* x4 = reinterpret_cast<float4*>(x);
    float4* m4 = reinterpret_cast<float4*>(m);
    float4* v4 = reinterpret_cast<float4*>(v);
    for (uint32_t base = 0; base < n4; base += NT * U) {
        float4 G[U], X[U], M[U], V[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n4) { G[u] = ld_stream(g4 + i); X[u] = ld_stream(x4 + i);
                          M[u] = ld_stream(m4 + i); V[u] = ld_stream(v4 + i); }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n4) {
                PALSGD_FOR4(adamw_elem(compv(G[u], c), comp(X[u], c), comp(M[u], c), comp(V[u], c), s))
                st_stream(x4 + i, X[u]); st_stream(m4 + i, M[u]); st_stream(v4 + i, V[u]);
            }
        }
    }
    const uint32_t i = (n4 << 2) + tid;
    if (i < len) { float xi = x[i], mi = m[i], vi = v[i]; adamw_elem(g[i], xi, mi, vi, s);
                   x[i] = xi; m[i] = mi; v[i] = vi; }
}

template <int U, int NT>
__device__ __forceinline__ void sgdm_chunk_f32(uint32_t tid, const float* __restrict__ g, float* __restrict__ x,
                                               float* __restrict__ buf, uint32_t len, const SgdScalars& s)
{
    const uint32_t n4 = len >> 2;
    const float4* g4 = reinterpret_cast<const float4*>(g);
    float4* x4 = reinterpret_cast<float4*>(x);
    float4* b4 = reinterpret_cast<float4*>(buf);
    for (uint32_t base = 0; base < n4; base += NT * U) {
        float4 G[U], X[U], B[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n4) { G[u] = ld_stream(g4 + i); X[u] = ld_stream(x4 + i); B[u] = ld_stream(b4 + i); }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n4) {
                PALSGD_FOR4(sgdm_elem(compv(G[u], c), comp(X[u], c), comp(B[u], c), s))
                st_stream(x4 + i, X[u]); st_stream(b4 + i, B[u]);
            }
        }
    }
    const uint32_t i = (n4 << 2) + tid;
    if (i < len) { float xi = x[i], bi = buf[i]; sgdm_elem(g[i], xi, bi, s); x[i] = xi; buf[i] = bi; }
}

// x_g is read with the default policy: slots that pull in the same step share it through L2.
template <int U, int NT>
__device__ __forceinline__ void pull_chunk_f32(uint32_t tid, float* __restrict__ x, const float* __restrict__ xg,
                                               uint32_t len, float beta)
{
    const uint32_t n4 = len >> 2;
    float4* x4 = reinterpret_cast<float4*>(x);
    const float4* q4 = reinterpret_cast<const float4*>(xg);
    for (uint32_t base = 0; base < n4; base += NT * U) {
        float4 X[U], Q[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n4) { X[u] = ld_stream(x4 + i); Q[u] = __ldg(q4 + i); }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n4) {
                PALSGD_FOR4(comp(X[u], c) = pull_elem(compv(X[u], c), compv(Q[u], c), beta))
                st_stream(x4 + i, X[u]);
            }
        }
    }
    const uint32_t i = (n4 << 2) + tid;
    if (i < len) x[i] = pull_elem(x[i], xg[i], beta);
}


// ---------------------------------------------------------------- bf16 + fp32-master chunk bodies
// Groups of 8 elements: one 128-bit load of bf16 gradients, two per fp32 stream.

__device__ __forceinline__ void unpack8(const uint4& h, float (&f)[8])
{
    f[0] = bf16_bits_to_f32(h.x & 0xFFFFu); f[1] = __uint_as_float(h.x & 0xFFFF0000u);
    f[2] = bf16_bits_to_f32(h.y & 0xFFFFu); f[3] = __uint_as_float(h.y & 0xFFFF0000u);
    f[4] = bf16_bits_to_f32(h.z & 0xFFFFu); f[5] = __uint_as_float(h.z & 0xFFFF0000u);
    f[6] = bf16_bits_to_f32(h.w & 0xFFFFu); f[7] = __uint_as_float(h.w & 0xFFFF0000u);
}

__device__ __forceinline__ uint4 pack8(const float4& a, const float4& b)
{
    return make_uint4(pack_bf16x2(a.x, a.y), pack_bf16x2(a.z, a.w),
                      pack_bf16x2(b.x, b.y), pack_bf16x2(b.z, b.w));
}

template <int U, int NT>
__device__ __forceinline__ void adamw_chunk_bf16(uint32_t tid, const __nv_bfloat16* __restrict__ g,
                                                 __nv_bfloat16* __restrict__ w, float* __restrict__ x,
                                                 float* __restrict__ m, float* __restrict__ v,
                                                 uint32_t len, const AdamScalars& s)
{
    const uint32_t n8 = len >> 3;
    const uint4* g8 = reinterpret_cast<const uint4*>(g);
    uint4* w8 = reinterpret_cast<uint4*>(w);
    float4* x4 = reinterpret_cast<float4*>(x);
    float4* m4 = reinterpret_cast<float4*>(m);
    float4* v4 = reinterpret_cast<float4*>(v);
    for (uint32_t base = 0; base < n8; base += NT * U) {
        uint4 G[U]; float4 X[U][2], M[U][2], V[U][2];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n8) {
                G[u] = ld_stream(g8 + i);
                X[u][0] = ld_stream(x4 + 2 * i); X[u][1] = ld_stream(x4 + 2 * i + 1);
                M[u][0] = ld_stream(m4 + 2 * i); M[u][1] = ld_stream(m4 + 2 * i + 1);
                V[u][0] = ld_stream(v4 + 2 * i); V[u][1] = ld_stream(v4 + 2 * i + 1);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n8) {
                float gf[8]; unpack8(G[u], gf);
                PALSGD_FOR4(adamw_elem(gf[c],     comp(X[u][0], c), comp(M[u][0], c), comp(V[u][0], c), s))
                PALSGD_FOR4(adamw_elem(gf[4 + c], comp(X[u][1], c), comp(M[u][1], c), comp(V[u][1], c), s))
                st_stream(x4 + 2 * i, X[u][0]); st_stream(x4 + 2 * i + 1, X[u][1]);
                st_stream(m4 + 2 * i, M[u][0]); st_stream(m4 + 2 * i + 1, M[u][1]);
                st_stream(v4 + 2 * i, V[u][0]); st_stream(v4 + 2 * i + 1, V[u][1]);
                st_stream(w8 + i, pack8(X[u][0], X[u][1]));
            }
        }
    }
    const uint32_t i = (n8 << 3) + tid;
    if (i < len) { float xi = x[i], mi = m[i], vi = v[i];
                   adamw_elem(__bfloat162float(g[i]), xi, mi, vi, s);
                   x[i] = xi; m[i] = mi; v[i] = vi; w[i] = __float2bfloat16_rn(xi); }
}

template <int U, int NT>
__device__ __forceinline__ void sgdm_chunk_bf16(uint32_t tid, const __nv_bfloat16* __restrict__ g,
                                                __nv_bfloat16* __restrict__ w, float* __restrict__ x,
                                                float* __restrict__ buf, uint32_t len, const SgdScalars& s)
{
    const uint32_t n8 = len >> 3;
    const uint4* g8 = reinterpret_cast<const uint4*>(g);
    uint4* w8 = reinterpret_cast<uint4*>(w);
    float4* x4 = reinterpret_cast<float4*>(x);
    float4* b4 = reinterpret_cast<float4*>(buf);
    for (uint32_t base = 0; base < n8; base += NT * U) {
        uint4 G[U]; float4 X[U][2], B[U][2];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n8) {
                G[u] = ld_stream(g8 + i);
                X[u][0] = ld_stream(x4 + 2 * i); X[u][1] = ld_stream(x4 + 2 * i + 1);
                B[u][0] = ld_stream(b4 + 2 * i); B[u][1] = ld_stream(b4 + 2 * i + 1);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n8) {
                float gf[8]; unpack8(G[u], gf);
                PALSGD_FOR4(sgdm_elem(gf[c],     comp(X[u][0], c), comp(B[u][0], c), s))
                PALSGD_FOR4(sgdm_elem(gf[4 + c], comp(X[u][1], c), comp(B[u][1], c), s))
                st_stream(x4 + 2 * i, X[u][0]); st_stream(x4 + 2 * i + 1, X[u][1]);
                st_stream(b4 + 2 * i, B[u][0]); st_stream(b4 + 2 * i + 1, B[u][1]);
                st_stream(w8 + i, pack8(X[u][0], X[u][1]));
            }
        }
    }
    const uint32_t i = (n8 << 3) + tid;
    if (i < len) { float xi = x[i], bi = buf[i]; sgdm_elem(__bfloat162float(g[i]), xi, bi, s);
                   x[i] = xi; buf[i] = bi; w[i] = __float2bfloat16_rn(xi); }
}

template <int U, int NT>
__device__ __forceinline__ void pull_chunk_bf16(uint32_t tid, __nv_bfloat16* __restrict__ w, float* __restrict__ x,
                                                const float* __restrict__ xg, uint32_t len, float beta)
{
    const uint32_t n8 = len >> 3;
    uint4* w8 = reinterpret_cast<uint4*>(w);
    float4* x4 = reinterpret_cast<float4*>(x);
    const float4* q4 = reinterpret_cast<const float4*>(xg);
    for (uint32_t base = 0; base < n8; base += NT * U) {
        float4 X[U][2], Q[U][2];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n8) { X[u][0] = ld_stream(x4 + 2 * i); X[u][1] = ld_stream(x4 + 2 * i + 1);
                          Q[u][0] = __ldg(q4 + 2 * i);      Q[u][1] = __ldg(q4 + 2 * i + 1); }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t i = base + u * NT + tid;
            if (i < n8) {
                PALSGD_FOR4(comp(X[u][0], c) = pull_elem(compv(X[u][0], c), compv(Q[u][0], c), beta))
                PALSGD_FOR4(comp(X[u][1], c) = pull_elem(compv(X[u][1], c), compv(Q[u][1], c), beta))
                st_stream(x4 + 2 * i, X[u][0]); st_stream(x4 + 2 * i + 1, X[u][1]);
                st_stream(w8 + i, pack8(X[u][0], X[u][1]));
            }
        }
    }
    const uint32_t i = (n8 << 3) + tid;
    if (i < len) { const float xi = pull_elem(x[i], xg[i], beta); x[i] = xi; w[i] = __float2bfloat16_rn(xi); }
}


// 4-element groups of bf16 values (64-bit accesses), used where a thread owns one 128-bit fp32 position
__device__ __forceinline__ void unpack4(const uint2& h, float (&f)[4])
{
    f[0] = bf16_bits_to_f32(h.x & 0xFFFFu); f[1] = __uint_as_float(h.x & 0xFFFF0000u);
    f[2] = bf16_bits_to_f32(h.y & 0xFFFFu); f[3] = __uint_as_float(h.y & 0xFFFF0000u);
}
__device__ __forceinline__ uint2 pack4(const float4& a)
{
    return make_uint2(pack_bf16x2(a.x, a.y), pack_bf16x2(a.z, a.w));
}

// ---------------------------------------------------------------- scalar bodies (unaligned segments)

template <int INNER, int PREC, int NT>
__device__ __forceinline__ void grad_chunk_scalar(uint32_t tid, const void* g, __nv_bfloat16* w, float* x, float* m, float* v,
                                                  uint32_t len, const AdamScalars& as, const SgdScalars& ss)
{
    for (uint32_t i = tid; i < len; i += NT) {
        const float gi = PREC ? __bfloat162float(static_cast<const __nv_bfloat16*>(g)[i])
                              : static_cast<const float*>(g)[i];
        float xi = x[i], mi = m[i];
        if (INNER == 0) { float vi = v[i]; adamw_elem(gi, xi, mi, vi, as); v[i] = vi; }
        else            { sgdm_elem(gi, xi, mi, ss); }
        x[i] = xi; m[i] = mi;
        if (PREC) w[i] = __float2bfloat16_rn(xi);
    }
}

template <int PREC, int NT>
__device__ __forceinline__ void pull_chunk_scalar(uint32_t tid, __nv_bfloat16* w, float* x, const float* xg, uint32_t len, float beta)
{
    for (uint32_t i = tid; i < len; i += NT) {
        const float xi = pull_elem(x[i], xg[i], beta);
        x[i] = xi;
        if (PREC) w[i] = __float2bfloat16_rn(xi);
    }
}

// ---------------------------------------------------------------- dispatch of one work item

template <int PREC, int U, int NT>
__device__ __forceinline__ void pull_item(uint32_t tid, const Tables& tb, uint32_t k, const Chunk& ch, float beta)
{
    const uint32_t seg = ch.seg & ~kSegVecFlag;
    const size_t   pi  = (size_t)k * tb.n_seg + seg;
    float* x = tb.xf[pi] + ch.off;
    const float* xg = tb.global[seg] + ch.off;
    __nv_bfloat16* w = PREC ? tb.xw[pi] + ch.off : nullptr;
    if (ch.seg & kSegVecFlag) {
        if (PREC) pull_chunk_bf16<U, NT>(tid, w, x, xg, ch.len, beta);
        else      pull_chunk_f32<U, NT>(tid, x, xg, ch.len, beta);
    } else {
        pull_chunk_scalar<PREC, NT>(tid, w, x, xg, ch.len, beta);
    }
}

template <int INNER, int PREC, int U, int NT>
__device__ __forceinline__ void grad_item(uint32_t tid, const Tables& tb, uint32_t k, const Chunk& ch,
                                          const AdamScalars& as, const SgdScalars& ss)
{
    const uint32_t seg = ch.seg & ~kSegVecFlag;
    const size_t   pi  = (size_t)k * tb.n_seg + seg;
    float* x = tb.xf[pi] + ch.off;
    float* m = tb.m[pi] + ch.off;
    float* v = INNER == 0 ? tb.v[pi] + ch.off : nullptr;
    if (PREC) {
        const __nv_bfloat16* g = static_cast<const __nv_bfloat16*>(tb.grad[pi]) + ch.off;
        __nv_bfloat16* w = tb.xw[pi] + ch.off;
        if (ch.seg & kSegVecFlag) {
            if (INNER == 0) adamw_chunk_bf16<U, NT>(tid, g, w, x, m, v, ch.len, as);
            else            sgdm_chunk_bf16<U, NT>(tid, g, w, x, m, ch.len, ss);
        } else {
            grad_chunk_scalar<INNER, 1, NT>(tid, g, w, x, m, v, ch.len, as, ss);
        }
    } else {
        const float* g = static_cast<const float*>(tb.grad[pi]) + ch.off;
        if (ch.seg & kSegVecFlag) {
            if (INNER == 0) adamw_chunk_f32<U, NT>(tid, g, x, m, v, ch.len, as);
            else            sgdm_chunk_f32<U, NT>(tid, g, x, m, ch.len, ss);
        } else {
            grad_chunk_scalar<INNER, 0, NT>(tid, g, nullptr, x, m, v, ch.len, as, ss);
        }
    }
}

// ---------------------------------------------------------------- fused inner step
// One launch per step of Algorithm 1's inner loop body.  Work item = (chunk c,
// worker k), k fastest, so neighbouring CTAs that pull share x_g through L2.
// Every CTA recomputes the K decisions of step t from the counter-based
// stream; the last CTA to finish advances the device counters.

template <int INNER, int PREC, int U, int MINB>
__global__ void __launch_bounds__(kThreads, MINB)
palsgd_inner_kernel(const __grid_constant__ InnerArgs a)
{
    __shared__ unsigned char s_pull[kMaxWorkers];
    __shared__ float s_bc1[kMaxWorkers], s_bc2[kMaxWorkers], s_clip[kMaxWorkers];

    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    DevState* st = tb.st;
    const unsigned long long t = st->t;

    if (threadIdx.x < K) {
        const uint32_t k = threadIdx.x;
        const bool pull = draw_pull(a.seed, t, a.k0 + k, a.thr);
        s_pull[k] = pull;
        s_clip[k] = a.clip_on ? st->clip[k] : 1.f;
        if (INNER == 0 && !pull) {                       // bias corrections for gradient step s_k + 1
            s_bc1[k] = (float)(1.0 - st->pow1[k] * a.beta1);
            s_bc2[k] = (float)(1.0 - st->pow2[k] * a.beta2);
        }
    }
    __syncthreads();

    // A step may be split into launches over disjoint worker ranges (gradients that arrive from the
    // host worker by worker); the last of them ticks the counters for all K workers.
    const uint32_t Kc = a.k_count;
    const uint64_t n_items = (uint64_t)tb.n_chunks * Kc;
    __shared__ unsigned int s_item;
    // a.dynamic: a grid of a few CTAs per SM draws items from a counter, so no CTA idles while others
    // still have a backlog; otherwise item = blockIdx.x, strided by the grid
    uint64_t item = blockIdx.x;
    if (a.dynamic) {
        if (threadIdx.x == 0) s_item = atomicAdd(&st->queue, 1u);
        __syncthreads();
        item = s_item;
    }
    while (item < n_items) {
        const uint32_t k = a.k_begin + (uint32_t)(item % Kc);
        const Chunk ch = tb.chunks[item / Kc];
        if (s_pull[k]) {
            pull_item<PREC, U, kThreads>(threadIdx.x, tb, k, ch, a.beta_pull);
        } else {
            const AdamScalars as{a.b1, a.b2, a.omb1, a.omb2, s_bc1[k], s_bc2[k], a.decay, a.lr, a.eps, s_clip[k]};
            const SgdScalars  ss{a.mu, a.wd, a.lr, s_clip[k]};
            grad_item<INNER, PREC, U, kThreads>(threadIdx.x, tb, k, ch, as, ss);
        }
        if (a.dynamic) {
            __syncthreads();                                   // everyone has read s_item
            if (threadIdx.x == 0) s_item = atomicAdd(&st->queue, 1u);
            __syncthreads();
            item = s_item;
        } else {
            item += gridDim.x;
        }
    }

    // ---- counter tick by the last CTA (all state reads above precede the atomic)
    __syncthreads();
    if (a.tick && threadIdx.x == 0) {
        __threadfence();
        const unsigned int prev = atomicAdd(&st->done, 1u);
        if (prev == gridDim.x - 1) {
            for (uint32_t k = 0; k < K; ++k) {
                const bool pull = s_pull[k];
                st->last_b[k] = pull;
                if (!pull) {
                    st->s[k] += 1;
                    if (INNER == 0) { st->pow1[k] *= a.beta1; st->pow2[k] *= a.beta2; }
                }
            }
            st->t = t + 1;
            st->done = 0;
            st->queue = 0;                                     // every CTA has drawn its last item by now
            __threadfence();
        }
    }
}

// ---------------------------------------------------------------- forced pull
template <int PREC, int U>
__global__ void __launch_bounds__(kThreads)
palsgd_pull_kernel(const __grid_constant__ PullArgs a)
{
    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    const uint64_t n_items = (uint64_t)tb.n_chunks * K;
    for (uint64_t item = blockIdx.x; item < n_items; item += gridDim.x) {
        const uint32_t k = (uint32_t)(item % K);
        if ((a.mask >> k) & 1ull) pull_item<PREC, U, kThreads>(threadIdx.x, tb, k, tb.chunks[item / K], a.beta);
    }
}

// ---------------------------------------------------------------- work distribution
// The outer-sync and DDP kernels walk an item table either strided by the grid or (dynamic) as a
// persistent grid that draws item indices from a counter in device memory.  The index of the NEXT
// item is requested once the current one has been computed (the atomic's round trip hides behind the
// fan-out of its results; requested earlier, in the middle of the load loop, the atomic kept the
// compiler from overlapping the loop's loads and cost the DDP kernel 15 %) and handed to the CTA
// through a two-slot mailbox in shared memory: slot (n+1)&1 is written during item n and read after
// the barrier that closes it, so one barrier per item orders everything.
struct ItemWalk {
    unsigned int* slots;        // two words of shared memory
    uint32_t      dynamic;
    DevState*     st;
    uint32_t      n;            // items done by this CTA
    unsigned int  pending;      // thread 0: the index requested for the next item

    __device__ __forceinline__ uint32_t first()
    {
        n = 0;
        if (threadIdx.x == 0) slots[0] = dynamic ? atomicAdd(&st->queue, 1u) : blockIdx.x;
        __syncthreads();
        return slots[0];
    }
    // call once the current item has been computed
    __device__ __forceinline__ void request_next(uint32_t cur)
    {
        if (threadIdx.x == 0) pending = dynamic ? atomicAdd(&st->queue, 1u) : cur + gridDim.x;
    }
    // call at the end of the item; contains the item's closing barrier
    __device__ __forceinline__ uint32_t next()
    {
        ++n;
        if (threadIdx.x == 0) slots[n & 1] = pending;
        __syncthreads();
        return slots[n & 1];
    }
};
// After the loop of a dynamic launch: the last CTA to finish rewinds the queue for the next launch.
__device__ __forceinline__ void rewind_queue(DevState* st)
{
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int prev = atomicAdd(&st->done, 1u);
        if (prev == gridDim.x - 1) { st->done = 0; st->queue = 0; __threadfence(); }
    }
}

// ---------------------------------------------------------------- bulk stores (TMA engine)
// One result written to K slots: the CTA stages it in shared memory once and a bulk
// asynchronous copy per slot and stream (cp.async.bulk shared -> global; this GPU's own
// memory, no multicast) carries it out, instead of K x 128-bit stores per thread.
// A persistent CTA alternates between two stage buffers: the copies of item n drain while
// item n+1 is loaded, computed and staged in the other buffer.  Bulk groups are per thread:
// every issuing thread commits exactly one group per item (an empty one if it has nothing to
// copy), so "all but the latest group have been read" means "the buffer of two items ago is free".
__device__ __forceinline__ void bulk_store(void* dst_gmem, const void* src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(__cvta_generic_to_global(dst_gmem)), "r"((uint32_t)__cvta_generic_to_shared(src_smem)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// shared memory of all groups but the latest `Pending` ones may be reused after this
template <int Pending>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(Pending) : "memory"); }
// generic-proxy writes to shared memory become visible to the asynchronous proxy
__device__ __forceinline__ void fence_async_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// ---------------------------------------------------------------- outer sync
// Per element: average of the K slots in ascending k, outer gradient, (Nesterov)
// momentum update, and the new global model written to x_g and to all K slots
// (and K bf16 working copies) in the same pass.

__device__ __forceinline__ float outer_elem(float sum, float Kf, float xg, float& u, float mu, float lr, int nesterov)
{
    const float xbar  = __fdiv_rn(sum, Kf);
    const float delta = __fsub_rn(xg, xbar);
    u = __fadd_rn(__fmul_rn(mu, u), delta);
    const float step = nesterov ? __fadd_rn(delta, __fmul_rn(mu, u)) : u;
    return __fsub_rn(xg, __fmul_rn(lr, step));
}

// OuterOPT = AdamW on the outer gradient: the inner optimizer's element formula with
// g = Delta, x = x_g, first moment u and second moment uv.
__device__ __forceinline__ float outer_elem_adamw(float sum, float Kf, float xg, float& u, float& uv, const AdamScalars& s)
{
    const float xbar  = __fdiv_rn(sum, Kf);
    const float delta = __fsub_rn(xg, xbar);
    adamw_elem(delta, xg, u, uv, s);
    return xg;
}

// OOPT: 0 = SGD with (Nesterov) momentum, 1 = AdamW (one more state stream).
// BCAST = 1: the new global model of a work item (with u and the bf16 copy) is staged in dynamic
// shared memory (8 (+4) (+2) bytes per element, sub_elems elements per buffer) and written to x_g,
// u and the K slots by bulk asynchronous stores; 16-byte-aligned pieces only, the rest takes the
// register path.
// SUMIN = 1: the sum over the workers is not formed here but read from the exchange buffer (it was
// formed by palsgd_outer_partial_kernel on every GPU and all-reduced), and Kf is the number of workers
// of the whole job; this launch then finishes the synchronisation for the local slots.
// B: slot loads issued together.  8 for K >= 5 (64 registers, 4 CTAs per SM); 4 for K <= 4, where half the
// registers for loads allow 5 CTAs per SM (K = 4, P = 2^24: 0.97 of the copy rate against 0.92).
template <int PREC, int OOPT, int BCAST, int SUMIN = 0, int B = 8>
__global__ void __launch_bounds__(kThreads, (BCAST && !OOPT) ? (B == 4 ? 5 : 4) : 1)
palsgd_outer_kernel(const __grid_constant__ OuterArgs a)
{
    extern __shared__ __align__(128) unsigned char outer_stage[];
    const AdamScalars os{a.ob1, a.ob2, a.oomb1, a.oomb2, a.obc1, a.obc2, a.odecay, a.lr, a.oeps};
    __shared__ float* s_x[kMaxWorkers];
    __shared__ __nv_bfloat16* s_w[kMaxWorkers];
    __shared__ unsigned int s_slots[2];
    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    const uint32_t stage_bytes = a.sub_elems * (8u + (OOPT ? 4u : 0u) + (PREC ? 2u : 0u));
    const bool issuer = BCAST && threadIdx.x <= K;         // thread k < K: slot k's copies; thread K: x_g and u

    ItemWalk walk{s_slots, a.dynamic, tb.st, 0, 0};
    for (uint32_t item = walk.first(); item < a.n_items; item = walk.next()) {
        const Chunk ch = a.items[item];
        const uint32_t seg = ch.seg & ~kSegVecFlag;
        // the stage buffer about to be refilled was handed to the copy engine two items ago
        if (issuer) { if (a.n_stage > 1) bulk_wait_read<1>(); else bulk_wait_read<0>(); }
        if (threadIdx.x < K) {                             // (the previous item's closing barrier protects s_x)
            const size_t pi = (size_t)threadIdx.x * tb.n_seg + seg;
            s_x[threadIdx.x] = tb.xf[pi] + ch.off;
            if (PREC) s_w[threadIdx.x] = tb.xw[pi] + ch.off;
        }
        __syncthreads();
        float* xg = tb.global[seg] + ch.off;
        float* um = tb.outer_mom[seg] + ch.off;
        float* uv = OOPT ? tb.outer_v[seg] + ch.off : nullptr;
        const float* sum_src = SUMIN ? a.sum_in + tb.exch_off[seg] + ch.off : nullptr;
        unsigned char* stage = outer_stage + (BCAST ? (walk.n % a.n_stage) * stage_bytes : 0u);
        float* sx = reinterpret_cast<float*>(stage);
        float* su = sx + a.sub_elems;

        uint32_t done = 0;
        if (ch.seg & kSegVecFlag) {
            const uint32_t n4 = ch.len >> 2;
            for (uint32_t i = threadIdx.x; i < n4; i += kThreads) {
                const float4 Q = __ldcs(reinterpret_cast<const float4*>(xg) + i);
                float4 Um = __ldcs(reinterpret_cast<const float4*>(um) + i);
                float4 Uv = make_float4(0.f, 0.f, 0.f, 0.f);
                if (OOPT) Uv = __ldcs(reinterpret_cast<const float4*>(uv) + i);
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                if (SUMIN) {
                    // the exchange buffer packs the tensors back to back: a piece may sit off 16-byte alignment there
                    if ((reinterpret_cast<uintptr_t>(sum_src) & 15u) == 0)
                        acc = __ldcs(reinterpret_cast<const float4*>(sum_src) + i);
                    else
                        acc = make_float4(__ldcs(sum_src + 4 * i), __ldcs(sum_src + 4 * i + 1),
                                          __ldcs(sum_src + 4 * i + 2), __ldcs(sum_src + 4 * i + 3));
                }
                for (uint32_t k0 = 0; !SUMIN && k0 < K; k0 += B) {
                    float4 R[B];
#pragma unroll
                    for (int j = 0; j < B; ++j)
                        if (k0 + j < K) R[j] = __ldcs(reinterpret_cast<const float4*>(s_x[k0 + j]) + i);
#pragma unroll
                    for (int j = 0; j < B; ++j)
                        if (k0 + j < K) {
                            if (k0 + j == 0) acc = R[j];
                            else { acc.x = __fadd_rn(acc.x, R[j].x); acc.y = __fadd_rn(acc.y, R[j].y);
                                   acc.z = __fadd_rn(acc.z, R[j].z); acc.w = __fadd_rn(acc.w, R[j].w); }
                        }
                }
                float4 N;
                if (OOPT) {
                    N.x = outer_elem_adamw(acc.x, a.Kf, Q.x, Um.x, Uv.x, os);
                    N.y = outer_elem_adamw(acc.y, a.Kf, Q.y, Um.y, Uv.y, os);
                    N.z = outer_elem_adamw(acc.z, a.Kf, Q.z, Um.z, Uv.z, os);
                    N.w = outer_elem_adamw(acc.w, a.Kf, Q.w, Um.w, Uv.w, os);
                } else {
                    N.x = outer_elem(acc.x, a.Kf, Q.x, Um.x, a.mu, a.lr, a.nesterov);
                    N.y = outer_elem(acc.y, a.Kf, Q.y, Um.y, a.mu, a.lr, a.nesterov);
                    N.z = outer_elem(acc.z, a.Kf, Q.z, Um.z, a.mu, a.lr, a.nesterov);
                    N.w = outer_elem(acc.w, a.Kf, Q.w, Um.w, a.mu, a.lr, a.nesterov);
                }
                if (BCAST) {
                    // x_g and u have one destination each and are written once the fan-out below has
                    // been fixed (a group of 4 left over by the bf16 16-byte rule is redone by the
                    // scalar loop from unmodified inputs), so they are staged too
                    reinterpret_cast<float4*>(sx)[i] = N;
                    reinterpret_cast<float4*>(su)[i] = Um;
                    if (OOPT) reinterpret_cast<float4*>(su + a.sub_elems)[i] = Uv;
                    if (PREC) reinterpret_cast<uint2*>(su + (OOPT ? 2 : 1) * a.sub_elems)[i] =
                                  make_uint2(pack_bf16x2(N.x, N.y), pack_bf16x2(N.z, N.w));
                    continue;
                }
                if (OOPT) __stcs(reinterpret_cast<float4*>(uv) + i, Uv);
                __stcs(reinterpret_cast<float4*>(xg) + i, N);
                __stcs(reinterpret_cast<float4*>(um) + i, Um);
                for (uint32_t k = 0; k < K; ++k) __stcs(reinterpret_cast<float4*>(s_x[k]) + i, N);
                if (PREC) {
                    const uint2 h = make_uint2(pack_bf16x2(N.x, N.y), pack_bf16x2(N.z, N.w));
                    for (uint32_t k = 0; k < K; ++k) __stcs(reinterpret_cast<uint2*>(s_w[k]) + i, h);
                }
            }
            done = n4 << 2;
            if (BCAST) done = PREC ? (done & ~7u) : done;       // whole 16-byte units of every stream
        }
        walk.request_next(item);                            // its round trip hides behind the fan-out below
        if (BCAST) {
            fence_async_shared();
            __syncthreads();
            if (issuer) {
                if (done > 0) {
                    if (threadIdx.x == K) {
                        bulk_store(xg, sx, done * 4);
                        bulk_store(um, su, done * 4);
                        if (OOPT) bulk_store(uv, su + a.sub_elems, done * 4);
                    } else {
                        bulk_store(s_x[threadIdx.x], sx, done * 4);
                        if (PREC) bulk_store(s_w[threadIdx.x], su + (OOPT ? 2 : 1) * a.sub_elems, done * 2);
                    }
                }
                bulk_commit();                                  // one group per item, possibly empty
            }
        }
        for (uint32_t i = done + threadIdx.x; i < ch.len; i += kThreads) {
            float sum = SUMIN ? sum_src[i] : s_x[0][i];
            for (uint32_t k = 1; !SUMIN && k < K; ++k) sum = __fadd_rn(sum, s_x[k][i]);
            float ui = um[i], xn;
            if (OOPT) { float vi = uv[i]; xn = outer_elem_adamw(sum, a.Kf, xg[i], ui, vi, os); uv[i] = vi; }
            else      { xn = outer_elem(sum, a.Kf, xg[i], ui, a.mu, a.lr, a.nesterov); }
            xg[i] = xn; um[i] = ui;
            for (uint32_t k = 0; k < K; ++k) s_x[k][i] = xn;
            if (PREC) { const __nv_bfloat16 h = __float2bfloat16_rn(xn);
                        for (uint32_t k = 0; k < K; ++k) s_w[k][i] = h; }
        }
    }
    if (issuer) bulk_wait_read<0>();                            // shared memory must outlive the copies' reads
    if (a.dynamic) rewind_queue(tb.st);
}

// ---------------------------------------------------------------- outer sync over several GPUs, first half
// Algorithm 1's All-Reduce when the K workers are spread over several GPUs: every GPU adds up its
// local workers' models in ascending local index and leaves the sum in the exchange buffer; the
// buffers are then summed across GPUs by the caller's collective, and palsgd_outer_kernel<.., SUMIN>
// divides by the job's worker count and finishes (Eq. (3), Eq. (4), restart of the local slots).
template <int B = 8>                                       // B: slot loads issued together
__global__ void __launch_bounds__(kThreads)
palsgd_outer_partial_kernel(const __grid_constant__ OuterArgs a)
{
    __shared__ float* s_x[kMaxWorkers];
    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    for (uint32_t item = blockIdx.x; item < a.n_items; item += gridDim.x) {
        const Chunk ch = a.items[item];
        const uint32_t seg = ch.seg & ~kSegVecFlag;
        __syncthreads();
        if (threadIdx.x < K) s_x[threadIdx.x] = tb.xf[(size_t)threadIdx.x * tb.n_seg + seg] + ch.off;
        __syncthreads();
        float* out = a.sum_out + tb.exch_off[seg] + ch.off;
        uint32_t done = 0;
        if (ch.seg & kSegVecFlag) {
            const uint32_t n4 = ch.len >> 2;
            for (uint32_t i = threadIdx.x; i < n4; i += kThreads) {
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (uint32_t k0 = 0; k0 < K; k0 += B) {
                    float4 R[B];
#pragma unroll
                    for (int j = 0; j < B; ++j)
                        if (k0 + j < K) R[j] = __ldcs(reinterpret_cast<const float4*>(s_x[k0 + j]) + i);
#pragma unroll
                    for (int j = 0; j < B; ++j)
                        if (k0 + j < K) {
                            if (k0 + j == 0) acc = R[j];
                            else { acc.x = __fadd_rn(acc.x, R[j].x); acc.y = __fadd_rn(acc.y, R[j].y);
                                   acc.z = __fadd_rn(acc.z, R[j].z); acc.w = __fadd_rn(acc.w, R[j].w); }
                        }
                }
                // (read again soon by the collective: default cache policy; the exchange buffer packs the
                //  tensors back to back, so a piece may sit off 16-byte alignment there)
                if ((reinterpret_cast<uintptr_t>(out) & 15u) == 0) reinterpret_cast<float4*>(out)[i] = acc;
                else { out[4 * i] = acc.x; out[4 * i + 1] = acc.y; out[4 * i + 2] = acc.z; out[4 * i + 3] = acc.w; }
            }
            done = n4 << 2;
        }
        for (uint32_t i = done + threadIdx.x; i < ch.len; i += kThreads) {
            float sum = s_x[0][i];
            for (uint32_t k = 1; k < K; ++k) sum = __fadd_rn(sum, s_x[k][i]);
            out[i] = sum;
        }
    }
}

// DDP warm-up phase with the workers spread over several GPUs, first half: the local workers' gradients
// added up in ascending local index (bf16 gradients widened exactly) into the exchange buffer.
template <int PREC, int B = 8>
__global__ void __launch_bounds__(kThreads)
palsgd_ddp_partial_kernel(const __grid_constant__ DdpArgs a)
{
    __shared__ const void* s_g[kMaxWorkers];
    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    for (uint32_t item = blockIdx.x; item < a.n_items; item += gridDim.x) {
        const Chunk ch = a.items[item];
        const uint32_t seg = ch.seg & ~kSegVecFlag;
        __syncthreads();
        if (threadIdx.x < K) {
            const size_t pi = (size_t)threadIdx.x * tb.n_seg + seg;
            if (PREC) s_g[threadIdx.x] = static_cast<const __nv_bfloat16*>(tb.grad[pi]) + ch.off;
            else      s_g[threadIdx.x] = static_cast<const float*>(tb.grad[pi]) + ch.off;
        }
        __syncthreads();
        float* out = a.sum_out + tb.exch_off[seg] + ch.off;
        uint32_t done = 0;
        if (ch.seg & kSegVecFlag) {
            const uint32_t n4 = ch.len >> 2;
            for (uint32_t i = threadIdx.x; i < n4; i += kThreads) {
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (uint32_t k0 = 0; k0 < K; k0 += B) {
                    float4 R[PREC ? 1 : B]; uint2 H[PREC ? B : 1];
#pragma unroll
                    for (int j = 0; j < B; ++j)
                        if (k0 + j < K) {
                            if (PREC) H[j] = __ldcs(static_cast<const uint2*>(s_g[k0 + j]) + i);
                            else      R[j] = __ldcs(static_cast<const float4*>(s_g[k0 + j]) + i);
                        }
#pragma unroll
                    for (int j = 0; j < B; ++j)
                        if (k0 + j < K) {
                            float4 r;
                            if (PREC) { float f[4]; unpack4(H[j], f); r = make_float4(f[0], f[1], f[2], f[3]); }
                            else      { r = R[j]; }
                            if (k0 + j == 0) acc = r;
                            else { acc.x = __fadd_rn(acc.x, r.x); acc.y = __fadd_rn(acc.y, r.y);
                                   acc.z = __fadd_rn(acc.z, r.z); acc.w = __fadd_rn(acc.w, r.w); }
                        }
                }
                if ((reinterpret_cast<uintptr_t>(out) & 15u) == 0) reinterpret_cast<float4*>(out)[i] = acc;
                else { out[4 * i] = acc.x; out[4 * i + 1] = acc.y; out[4 * i + 2] = acc.z; out[4 * i + 3] = acc.w; }
            }
            done = n4 << 2;
        }
        for (uint32_t i = done + threadIdx.x; i < ch.len; i += kThreads) {
            float sum = 0.f;
            for (uint32_t k = 0; k < K; ++k) {
                const float gk = PREC ? __bfloat162float(static_cast<const __nv_bfloat16*>(s_g[k])[i])
                                      : static_cast<const float*>(s_g[k])[i];
                sum = k == 0 ? gk : __fadd_rn(sum, gk);
            }
            out[i] = sum;
        }
    }
}

// Initialisation when the workers are spread over several GPUs: x_g = (sum over ALL workers) / K_total,
// the sum having been formed by palsgd_outer_partial_kernel on every GPU and all-reduced.
template <int UNUSED = 0>
__global__ void __launch_bounds__(kThreads)
palsgd_global_from_sum_kernel(const __grid_constant__ OuterArgs a)
{
    const Tables& tb = a.tb;
    for (uint32_t item = blockIdx.x; item < a.n_items; item += gridDim.x) {
        const Chunk ch = a.items[item];
        const uint32_t seg = ch.seg & ~kSegVecFlag;
        const float* sum = a.sum_in + tb.exch_off[seg] + ch.off;
        float* xg = tb.global[seg] + ch.off;
        for (uint32_t i = threadIdx.x; i < ch.len; i += kThreads) xg[i] = __fdiv_rn(sum[i], a.Kf);
    }
}

// ---------------------------------------------------------------- DDP warm-up step
// Mini-batch phase that precedes Algorithm 1 (Sec. 3.3, Sec. 4.1): per element the K
// gradients are summed in ascending k and divided by K, ONE optimizer step is taken on
// worker 0's model and state with the plain step size alpha_t, and the result goes to
// every slot and to the global model copy.  Reads 4K+12 bytes (2K+12 with bf16
// gradients) and writes 12K+4 (14K+4) per parameter for AdamW: store-dominated.

// BCAST = 1: the new x, m, v (and bf16 copy) of a work item are staged in dynamic shared memory
// ((12 or 8) + 2 bytes per element, sub_elems elements per buffer) and written to the K slots and
// to x_g by bulk asynchronous stores; 16-byte-aligned pieces only, the rest takes the register path.
// SUMIN = 1: the gradient sum over ALL workers of a job comes ready-made from the exchange buffer
// (palsgd_ddp_partial_kernel on every GPU, then the caller's all-reduce) and Kf is the job's worker count.
template <int INNER, int PREC, int BCAST, int SUMIN = 0>
__global__ void __launch_bounds__(kThreads)
palsgd_ddp_kernel(const __grid_constant__ DdpArgs a)
{
    extern __shared__ __align__(128) unsigned char ddp_stage[];
    __shared__ float* s_x[kMaxWorkers];
    __shared__ float* s_m[kMaxWorkers];
    __shared__ float* s_v[kMaxWorkers];
    __shared__ const void* s_g[kMaxWorkers];
    __shared__ __nv_bfloat16* s_w[kMaxWorkers];
    __shared__ unsigned int s_slots[2];
    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    DevState* st = tb.st;
    constexpr int B = 8;                                   // gradient loads issued together
    const uint32_t stage_bytes = a.sub_elems * ((INNER == 0 ? 12u : 8u) + (PREC ? 2u : 0u));
    const bool issuer = BCAST && threadIdx.x <= K;         // thread k < K: slot k's copies; thread K: x_g

    // bias corrections for gradient step s_0 + 1 (all workers share worker 0's count in this phase)
    const unsigned long long t = st->t;
    AdamScalars as{a.b1, a.b2, a.omb1, a.omb2, 1.f, 1.f, a.decay, a.lr, a.eps};
    if (INNER == 0) {
        as.bc1 = (float)(1.0 - st->pow1[0] * a.beta1);
        as.bc2 = (float)(1.0 - st->pow2[0] * a.beta2);
    }
    SgdScalars ss{a.mu, a.wd, a.lr};
    if (a.clip_on) { as.clip = st->clip[0]; ss.clip = as.clip; }   // the clip applies to the averaged gradient

    ItemWalk walk{s_slots, a.dynamic, st, 0, 0};
    for (uint32_t item = walk.first(); item < a.n_items; item = walk.next()) {
        const Chunk ch = a.items[item];
        const uint32_t seg = ch.seg & ~kSegVecFlag;
        if (issuer) { if (a.n_stage > 1) bulk_wait_read<1>(); else bulk_wait_read<0>(); }
        if (threadIdx.x < K) {                             // (the previous item's closing barrier protects these)
            const size_t pi = (size_t)threadIdx.x * tb.n_seg + seg;
            s_x[threadIdx.x] = tb.xf[pi] + ch.off;
            s_m[threadIdx.x] = tb.m[pi] + ch.off;
            if (INNER == 0) s_v[threadIdx.x] = tb.v[pi] + ch.off;
            if (PREC) { s_w[threadIdx.x] = tb.xw[pi] + ch.off;
                        s_g[threadIdx.x] = static_cast<const __nv_bfloat16*>(tb.grad[pi]) + ch.off; }
            else      { s_g[threadIdx.x] = static_cast<const float*>(tb.grad[pi]) + ch.off; }
        }
        __syncthreads();
        float* xg = tb.global[seg] + ch.off;
        const float* sum_src = SUMIN ? a.sum_in + tb.exch_off[seg] + ch.off : nullptr;
        unsigned char* stage = ddp_stage + (BCAST ? (walk.n % a.n_stage) * stage_bytes : 0u);
        float* sx = reinterpret_cast<float*>(stage);
        float* sm = sx + a.sub_elems;
        float* sv = sm + a.sub_elems;

        uint32_t done = 0;
        if (ch.seg & kSegVecFlag) {
            const uint32_t n4 = ch.len >> 2;
            for (uint32_t i = threadIdx.x; i < n4; i += kThreads) {
                float4 X = __ldcs(reinterpret_cast<const float4*>(s_x[0]) + i);
                float4 M = __ldcs(reinterpret_cast<const float4*>(s_m[0]) + i);
                float4 V = make_float4(0.f, 0.f, 0.f, 0.f);
                if (INNER == 0) V = __ldcs(reinterpret_cast<const float4*>(s_v[0]) + i);
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                if (SUMIN) {
                    if ((reinterpret_cast<uintptr_t>(sum_src) & 15u) == 0)
                        acc = __ldcs(reinterpret_cast<const float4*>(sum_src) + i);
                    else
                        acc = make_float4(__ldcs(sum_src + 4 * i), __ldcs(sum_src + 4 * i + 1),
                                          __ldcs(sum_src + 4 * i + 2), __ldcs(sum_src + 4 * i + 3));
                }
                for (uint32_t k0 = 0; !SUMIN && k0 < K; k0 += B) {
                    // bf16 gradients stay packed in registers until they are added (half the registers)
                    float4 R[PREC ? 1 : B]; uint2 H[PREC ? B : 1];
#pragma unroll
                    for (int j = 0; j < B; ++j)
                        if (k0 + j < K) {
                            if (PREC) H[j] = __ldcs(static_cast<const uint2*>(s_g[k0 + j]) + i);
                            else      R[j] = __ldcs(static_cast<const float4*>(s_g[k0 + j]) + i);
                        }
#pragma unroll
                    for (int j = 0; j < B; ++j)
                        if (k0 + j < K) {
                            float4 r;
                            if (PREC) { float f[4]; unpack4(H[j], f); r = make_float4(f[0], f[1], f[2], f[3]); }
                            else      { r = R[j]; }
                            if (k0 + j == 0) acc = r;
                            else { acc.x = __fadd_rn(acc.x, r.x); acc.y = __fadd_rn(acc.y, r.y);
                                   acc.z = __fadd_rn(acc.z, r.z); acc.w = __fadd_rn(acc.w, r.w); }
                        }
                }
                float4 G;
                G.x = __fdiv_rn(acc.x, a.Kf); G.y = __fdiv_rn(acc.y, a.Kf);
                G.z = __fdiv_rn(acc.z, a.Kf); G.w = __fdiv_rn(acc.w, a.Kf);
                if (INNER == 0) { PALSGD_FOR4(adamw_elem(compv(G, c), comp(X, c), comp(M, c), comp(V, c), as)) }
                else            { PALSGD_FOR4(sgdm_elem(compv(G, c), comp(X, c), comp(M, c), ss)) }
                if (BCAST) {                                // stage; the fan-out follows the loop
                    reinterpret_cast<float4*>(sx)[i] = X;
                    reinterpret_cast<float4*>(sm)[i] = M;
                    if (INNER == 0) reinterpret_cast<float4*>(sv)[i] = V;
                    if (PREC) reinterpret_cast<uint2*>(sm + (INNER == 0 ? 2 : 1) * a.sub_elems)[i] = pack4(X);
                    continue;
                }
                __stcs(reinterpret_cast<float4*>(xg) + i, X);
                for (uint32_t k = 0; k < K; ++k) {
                    __stcs(reinterpret_cast<float4*>(s_x[k]) + i, X);
                    __stcs(reinterpret_cast<float4*>(s_m[k]) + i, M);
                    if (INNER == 0) __stcs(reinterpret_cast<float4*>(s_v[k]) + i, V);
                }
                if (PREC) {
                    const uint2 h = pack4(X);
                    for (uint32_t k = 0; k < K; ++k) __stcs(reinterpret_cast<uint2*>(s_w[k]) + i, h);
                }
            }
            done = n4 << 2;
            // whole 16-byte units only: the bf16 stream needs a multiple of 8 elements; what is left
            // of an odd group of 4 is redone below by the scalar loop (its inputs are still intact)
            if (BCAST) done = PREC ? (done & ~7u) : done;
        }
        walk.request_next(item);                            // its round trip hides behind the fan-out below
        if (BCAST) {
            fence_async_shared();
            __syncthreads();
            if (issuer) {
                if (done > 0) {
                    if (threadIdx.x == K) {
                        bulk_store(xg, sx, done * 4);
                    } else {
                        const uint32_t k = threadIdx.x;
                        bulk_store(s_x[k], sx, done * 4);
                        bulk_store(s_m[k], sm, done * 4);
                        if (INNER == 0) bulk_store(s_v[k], sv, done * 4);
                        if (PREC) bulk_store(s_w[k], sm + (INNER == 0 ? 2 : 1) * a.sub_elems, done * 2);
                    }
                }
                bulk_commit();                                  // one group per item, possibly empty
            }
        }
        for (uint32_t i = done + threadIdx.x; i < ch.len; i += kThreads) {
            float sum = SUMIN ? sum_src[i] : 0.f;
            for (uint32_t k = 0; !SUMIN && k < K; ++k) {
                const float gk = PREC ? __bfloat162float(static_cast<const __nv_bfloat16*>(s_g[k])[i])
                                      : static_cast<const float*>(s_g[k])[i];
                sum = k == 0 ? gk : __fadd_rn(sum, gk);
            }
            const float g = __fdiv_rn(sum, a.Kf);
            float xi = s_x[0][i], mi = s_m[0][i], vi = 0.f;
            if (INNER == 0) { vi = s_v[0][i]; adamw_elem(g, xi, mi, vi, as); }
            else            { sgdm_elem(g, xi, mi, ss); }
            xg[i] = xi;
            for (uint32_t k = 0; k < K; ++k) {
                s_x[k][i] = xi; s_m[k][i] = mi;
                if (INNER == 0) s_v[k][i] = vi;
                if (PREC) s_w[k][i] = __float2bfloat16_rn(xi);
            }
        }
    }
    if (issuer) bulk_wait_read<0>();                            // shared memory must outlive the copies' reads

    // ---- counter tick by the last CTA (all state reads above precede the atomic)
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int prev = atomicAdd(&st->done, 1u);
        if (prev == gridDim.x - 1) {
            const unsigned long long s0 = st->s[0] + 1;
            const double p1 = INNER == 0 ? st->pow1[0] * a.beta1 : st->pow1[0];
            const double p2 = INNER == 0 ? st->pow2[0] * a.beta2 : st->pow2[0];
            for (uint32_t k = 0; k < K; ++k) {
                st->s[k] = s0; st->pow1[k] = p1; st->pow2[k] = p2; st->last_b[k] = 0;
            }
            st->t = t + 1;
            st->done = 0;
            st->queue = 0;
            __threadfence();
        }
    }
}

// ---------------------------------------------------------------- set-up
// x_g <- fixed-order mean of the slots, u <- 0, m, v <- 0, bf16 working <- RNE(master).
template <int PREC>
__global__ void __launch_bounds__(kThreads)
palsgd_init_kernel(const __grid_constant__ OuterArgs a, int has_v)
{
    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    for (uint32_t c = blockIdx.x; c < tb.n_chunks; c += gridDim.x) {
        const Chunk ch = tb.chunks[c];
        const uint32_t seg = ch.seg & ~kSegVecFlag;
        float* xg = tb.global[seg] + ch.off;
        float* um = tb.outer_mom[seg] + ch.off;
        float* uv = tb.outer_v ? tb.outer_v[seg] + ch.off : nullptr;
        for (uint32_t i = threadIdx.x; i < ch.len; i += kThreads) {
            if (uv) uv[i] = 0.f;
            float sum = 0.f;
            for (uint32_t k = 0; k < K; ++k) {
                const size_t pi = (size_t)k * tb.n_seg + seg;
                const float xi = tb.xf[pi][ch.off + i];
                sum = k == 0 ? xi : __fadd_rn(sum, xi);
                tb.m[pi][ch.off + i] = 0.f;
                if (has_v) tb.v[pi][ch.off + i] = 0.f;
                if (PREC) tb.xw[pi][ch.off + i] = __float2bfloat16_rn(xi);
            }
            xg[i] = __fdiv_rn(sum, a.Kf);
            um[i] = 0.f;
        }
    }
}

}  // namespace palsgd
