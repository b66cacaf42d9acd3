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
    double dn[2], up[2];        // two independent chains (even / odd element position), rounded down / up
    double ok[2];               // their (common) values at the start of the current piece

    __device__ __forceinline__ void init()
    {
#pragma unroll
        for (int j = 0; j < 2; ++j) { dn[j] = 0.0; up[j] = 0.0; ok[j] = 0.0; }
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
        const bool exact = dn[0] == up[0] && dn[1] == up[1];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            if (exact) ok[j] = dn[j];
            else { dn[j] = ok[j]; up[j] = ok[j]; }
        }
        return exact;
    }
};

// One piece of a work item of the norm pass: `len` bf16 gradients at g.
struct NormPiece { const void* g; uint32_t len; uint32_t vec; };
constexpr uint32_t kNormGroupMax = 8;      // chunks per work item at most
constexpr int kNormU = 4;                  // 128-bit loads per thread and piece

// First kThreads * kNormU groups of 8 of a 16-byte-aligned piece into registers (zeros elsewhere).
__device__ __forceinline__ void norm_piece_load(uint4 (&R)[kNormU], const NormPiece& p)
{
    const uint4* g8 = static_cast<const uint4*>(p.g);
    const uint32_t n8 = p.vec ? min(p.len >> 3, kThreads * (uint32_t)kNormU) : 0u;
#pragma unroll
    for (int u = 0; u < kNormU; ++u) {
        const uint32_t i = u * kThreads + threadIdx.x;
        R[u] = i < n8 ? ld_stream(g8 + i) : make_uint4(0u, 0u, 0u, 0u);            // zeros add nothing
    }
}

// The loaded groups into the fast chains; if the chains' test then fails, the chains are put back and
// the same elements are added once more in double-double (rare; the data is still in cache).  Whatever
// the registers did not cover (an unaligned piece, a piece longer than the registers, an odd tail)
// goes through the double-double accumulator as well.
__device__ __forceinline__ void norm_piece_consume(FastSq& f, DD& slow, const uint4 (&R)[kNormU], const NormPiece& p)
{
    const uint4* g8 = static_cast<const uint4*>(p.g);
    const uint32_t n8_all = p.vec ? p.len >> 3 : 0u;
    const uint32_t n8 = min(n8_all, kThreads * (uint32_t)kNormU);
#pragma unroll
    for (int u = 0; u < kNormU; ++u) {
        float v[8]; unpack8(R[u], v);
#pragma unroll
        for (int c = 0; c < 8; ++c) f.add(c & 1, v[c]);
    }
    uint32_t redo_from = n8;                                // groups [redo_from, n8_all) go the slow way
    if (!f.settle()) redo_from = 0;
    for (uint32_t i = redo_from + threadIdx.x; i < n8_all; i += kThreads) {
        float v[8]; unpack8(__ldg(g8 + i), v);
#pragma unroll
        for (int c = 0; c < 8; ++c) dd_square_in(slow, v[c]);
    }
    for (uint32_t i = (n8_all << 3) + threadIdx.x; i < p.len; i += kThreads)
        dd_square_in(slow, __bfloat162float(static_cast<const __nv_bfloat16*>(p.g)[i]));
}

// All pieces of a work item, software-pipelined: the loads of piece c+1 are in flight while piece c
// is being added up (the pieces' addresses were resolved beforehand, so nothing but the data itself
// is waited for).
__device__ __forceinline__ void norm_group_bf16_fast(FastSq& f, DD& slow, const NormPiece* pieces, uint32_t n)
{
    uint4 A[kNormU], B[kNormU];
    norm_piece_load(A, pieces[0]);
    for (uint32_t c = 0; c < n; c += 2) {
        if (c + 1 < n) norm_piece_load(B, pieces[c + 1]);
        norm_piece_consume(f, slow, A, pieces[c]);
        if (c + 2 < n) norm_piece_load(A, pieces[c + 2]);
        if (c + 1 < n) norm_piece_consume(f, slow, B, pieces[c + 1]);
    }
}

// ---- fp32 gradients: the same pipelining over pre-resolved pieces (of at most 4 * kThreads * kNormUf
// elements each), every square through the double-double accumulators.
constexpr int kNormUf = 4;                 // 128-bit loads per thread and piece, fp32 form (2: 0.148 against 0.125-0.137 ms on c2)
__device__ __forceinline__ void norm_piece_load_f32(float4 (&R)[kNormUf], const NormPiece& p)
{
    const float4* g4 = static_cast<const float4*>(p.g);
    const uint32_t n4 = p.vec ? min(p.len >> 2, kThreads * (uint32_t)kNormUf) : 0u;
#pragma unroll
    for (int u = 0; u < kNormUf; ++u) {
        const uint32_t i = u * kThreads + threadIdx.x;
        R[u] = i < n4 ? ld_stream(g4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);        // zeros add nothing
    }
}
__device__ __forceinline__ void norm_piece_consume_f32(DD (&q)[4], const float4 (&R)[kNormUf], const NormPiece& p)
{
#pragma unroll
    for (int u = 0; u < kNormUf; ++u) {
        dd_square_in(q[0], R[u].x); dd_square_in(q[1], R[u].y);
        dd_square_in(q[2], R[u].z); dd_square_in(q[3], R[u].w);
    }
    const uint32_t done = p.vec ? min(p.len >> 2, kThreads * (uint32_t)kNormUf) << 2 : 0u;
    for (uint32_t i = done + threadIdx.x; i < p.len; i += kThreads)     // unaligned pieces, odd tails
        dd_square_in(q[0], static_cast<const float*>(p.g)[i]);
}
__device__ __forceinline__ void norm_group_f32(DD (&q)[4], const NormPiece* pieces, uint32_t n)
{
    float4 A[kNormUf], B[kNormUf];
    norm_piece_load_f32(A, pieces[0]);
    for (uint32_t c = 0; c < n; c += 2) {
        if (c + 1 < n) norm_piece_load_f32(B, pieces[c + 1]);
        norm_piece_consume_f32(q, A, pieces[c]);
        if (c + 2 < n) norm_piece_load_f32(A, pieces[c + 2]);
        if (c + 1 < n) norm_piece_consume_f32(q, B, pieces[c + 1]);
    }
}

// One launch ahead of a step whose gradients are clipped.  The grid is persistent (a few CTAs per
// SM).  Every CTA works for ONE worker that takes a gradient step (ddp = 0), or for the one
// averaged gradient (ddp = 1: formed exactly as the DDP step forms it): with n_act such workers,
// CTA b serves the (b mod n_act)-th of them and walks over the groups of a.group consecutive
// chunks  b / n_act, b / n_act + C, ...  (C = gridDim / n_act CTAs per worker), adding up in
// registers across all of them, so that the CTA-wide reduction is paid once per CTA.  Every CTA
// leaves one double-double partial in tb.norm_part[b]; the last CTA to finish adds the partials
// of each worker (one warp per worker) and writes sumsq and the clip coefficient to the device
// state.  The sums are exact up to the final rounding, so the result does not depend on how the
// work was cut.
// DDP = 1: the one norm of the averaged gradient (DDP warm-up phase); 0: one norm per worker.
template <int PREC, int DDP>
__global__ void __launch_bounds__(kThreads, 3)
palsgd_gradnorm_kernel(const __grid_constant__ NormArgs a)
{
    __shared__ unsigned char s_act[kMaxWorkers];            // the workers that take a gradient step, ascending
    __shared__ unsigned int s_n_act;
    __shared__ DD s_warp[kThreads / 32];
    __shared__ const void* s_g[kMaxWorkers];
    __shared__ NormPiece s_piece[(kThreads / 32) * 4 * kNormGroupMax];
    __shared__ unsigned int s_last;
    const Tables& tb = a.tb;
    const uint32_t K = tb.K;
    DevState* st = tb.st;
    const unsigned long long t = st->t;

    if (threadIdx.x == 0) {
        unsigned int n = 0;
        if (DDP) { s_act[0] = 0; n = 1; }
        else for (uint32_t k = 0; k < K; ++k) if (!draw_pull(a.seed, t, a.k0 + k, a.thr)) s_act[n++] = (unsigned char)k;
        s_n_act = n;
    }
    __syncthreads();
    const uint32_t n_act = s_n_act;
    const uint32_t per_worker = n_act ? gridDim.x / n_act : 0u;        // CTAs per worker (the rest idle)
    const uint32_t mine = n_act ? blockIdx.x % n_act : 0u;
    const uint32_t lane_of_worker = n_act ? blockIdx.x / n_act : 0u;
    const bool working = n_act && lane_of_worker < per_worker;
    const uint32_t k = working ? s_act[mine] : 0u;

    const uint32_t n_groups = (tb.n_chunks + a.group - 1) / a.group;
    const size_t gsz = PREC ? 2 : 4;
    DD q[4] = {{0.0, 0.0}, {0.0, 0.0}, {0.0, 0.0}, {0.0, 0.0}};
    FastSq f; f.init();
    for (uint32_t grp = lane_of_worker; working && grp < n_groups; grp += per_worker) {
        const uint32_t c_begin = grp * a.group;
        const uint32_t c_end = min(c_begin + a.group, tb.n_chunks);
        if (PREC == 1 && !DDP) {
            // bf16 gradients: plain binary64 chains whose exactness is tested piece by piece.  The pieces'
            // addresses (chunk table -> pointer table, two dependent reads) are resolved for the whole
            // group at once, so that the data loads of successive pieces can overlap
            // (every warp resolves them for itself into its own slots: no CTA-wide barrier per group)
            NormPiece* my_piece = s_piece + (threadIdx.x >> 5) * (4 * kNormGroupMax);
            const uint32_t lane = threadIdx.x & 31;
            __syncwarp();                                   // the previous group's readers of my_piece
            if (lane < c_end - c_begin) {
                const Chunk ch = tb.chunks[c_begin + lane];
                const uint32_t seg = ch.seg & ~kSegVecFlag;
                my_piece[lane] = NormPiece{static_cast<const char*>(tb.grad[(size_t)k * tb.n_seg + seg]) + ch.off * gsz,
                                           ch.len, (ch.seg & kSegVecFlag) ? 1u : 0u};
            }
            __syncwarp();
            norm_group_bf16_fast(f, q[0], my_piece, c_end - c_begin);
            // the chains hold exact sums: fold them into the double-double total and start them afresh, so
            // that the running sums stay small (the smaller they are, the smaller the elements they take exactly)
            q[1] = dd_add(q[1], dd_add(DD{f.dn[0], 0.0}, DD{f.dn[1], 0.0}));
            f.init();
            continue;
        }
        if (PREC == 0 && !DDP) {
            // fp32 gradients: every chunk becomes pieces of at most 4096 elements (what one round of loads
            // covers), resolved per warp as above, then streamed with the next piece's loads in flight
            constexpr uint32_t kPieceElems = 4u * kThreads * kNormUf;
            const uint32_t per_chunk = (tb.chunk_elems + kPieceElems - 1) / kPieceElems;    // 1 or 2
            const uint32_t n_pieces = (c_end - c_begin) * per_chunk;
            if (n_pieces <= 4 * kNormGroupMax) {
                NormPiece* my_piece = s_piece + (threadIdx.x >> 5) * (4 * kNormGroupMax);
                const uint32_t lane = threadIdx.x & 31;
                __syncwarp();
                if (lane < n_pieces) {
                    const Chunk ch = tb.chunks[c_begin + lane / per_chunk];
                    const uint32_t seg = ch.seg & ~kSegVecFlag;
                    const uint32_t begin = (lane % per_chunk) * kPieceElems;
                    const uint32_t len = ch.len > begin ? min(ch.len - begin, kPieceElems) : 0u;
                    my_piece[lane] = NormPiece{static_cast<const char*>(tb.grad[(size_t)k * tb.n_seg + seg]) +
                                                   (ch.off + begin) * gsz, len, (ch.seg & kSegVecFlag) ? 1u : 0u};
                }
                __syncwarp();
                norm_group_f32(q, my_piece, n_pieces);
                continue;
            }
        }
        for (uint32_t c = c_begin; c < c_end; ++c) {
        const Chunk ch = tb.chunks[c];
        const uint32_t seg = ch.seg & ~kSegVecFlag;
        const bool vec = (ch.seg & kSegVecFlag) != 0;
        if (DDP) {
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
        } else {
            const char* g = static_cast<const char*>(tb.grad[(size_t)k * tb.n_seg + seg]) + ch.off * gsz;
            sumsq_chunk<PREC>(q, g, ch.len, vec);
        }
        }
    }
    const DD mine_tot = dd_block_sum(dd_add(dd_add(q[0], q[1]), dd_add(q[2], q[3])), s_warp);
    if (threadIdx.x == 0) tb.norm_part[blockIdx.x] = make_double2(mine_tot.hi, mine_tot.lo);

    // ---- the last CTA to finish adds the partials: warp w takes the workers w, w + 8, ...
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned int prev = atomicAdd(&st->done_norm, 1u);
        s_last = (prev == gridDim.x - 1);
        __threadfence();
    }
    __syncthreads();
    if (!s_last) return;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (uint32_t w = warp; w < n_act; w += kThreads / 32) {
        DD acc{0.0, 0.0};
        for (uint32_t j = lane; j < per_worker; j += 32) {   // CTA j * n_act + w worked for this worker
            const double2 p = __ldcg(tb.norm_part + (size_t)j * n_act + w);
            acc = dd_add(acc, DD{p.x, p.y});
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            DD o;
            o.hi = __shfl_down_sync(0xFFFFFFFFu, acc.hi, off);
            o.lo = __shfl_down_sync(0xFFFFFFFFu, acc.lo, off);
            acc = dd_add(acc, o);
        }
        if (lane == 0) {
            const double sumsq = isfinite(acc.hi) ? __dadd_rn(acc.hi, acc.lo) : acc.hi;
            const double coef = __ddiv_rn(a.max_norm, __dadd_rn(__dsqrt_rn(sumsq), 1e-6));
            const float clip = (float)(coef < 1.0 ? coef : 1.0);
            if (DDP) { for (uint32_t kk = 0; kk < K; ++kk) { st->sumsq[kk] = sumsq; st->clip[kk] = clip; } }
            else       { st->sumsq[s_act[w]] = sumsq; st->clip[s_act[w]] = clip; }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) { st->done_norm = 0; __threadfence(); }
}

}  // namespace palsgd
